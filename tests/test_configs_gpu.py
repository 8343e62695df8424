"""Parity at the full sizes of the benchmark configurations, on sampled steps and rows.

The oracle ingests every chunk (so its cache is the whole history in fp64) but evaluates only
sampled query rows: a row over a 131 072-token prefix costs ~2 GFLOP in fp64.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_12471_b200 import binding, workloads
from tests.chain import TOL, CacheBits, assert_chain_cache_bits, assert_within, run_chain, to_f64

pytestmark = pytest.mark.gpu


def _steps(n_steps, rng, extra=8):
    """Checked steps of a long chain: seven fixed ones and `extra` seeded-random ones."""
    fixed = {0, 1, 2, n_steps // 4, n_steps // 2, n_steps - 2, n_steps - 1}
    fixed = {s for s in fixed if 0 <= s < n_steps}
    fixed.update(int(x) for x in rng.integers(0, n_steps, size=extra))
    return sorted(fixed)


# rows of a checked step: six fixed ones (first two, the two around the middle, last two) and ten
# seeded-random ones (chain.sample_rows)
ROWS_EXTRA = 10


def test_config2_llama_16k_chunks_of_2048():
    w = workloads.LLAMA_16K
    chunks = [w.chunk] * w.n_steps
    res, cache, _, _ = run_chain(w, chunks, seed=21, rows_per_step=ROWS_EXTRA)
    assert len(cache) == 16384
    assert_within(res, "bf16", "config 2")
    # inputs are scaled by 1/sqrt(128): outputs are ~1e-3, so the relative error is the telling one
    assert res.rel_rms <= 2e-2, res.rel_rms
    # what the eight steps appended, every row of it
    bits = assert_chain_cache_bits(cache, w, chunks, seed=21, what="config 2 cache")
    assert bits.elements == 16384 * 8 * 128


def test_config3_deep_chain_128k_depth_511():
    """The benchmark's launch configuration: 512 steps of 256 tokens, prefix up to 130 816."""
    w = workloads.DEEP_CHAIN
    chunks = [w.chunk] * w.n_steps
    steps = _steps(w.n_steps, np.random.default_rng(3))
    res, cache, _, _ = run_chain(w, chunks, seed=22, check_steps=steps, rows_per_step=ROWS_EXTRA)
    assert len(cache) == 131072 == 512 * 256
    assert_within(res, "bf16", "config 3")
    assert res.rel_rms <= 2e-2, res.rel_rms
    print("config3 drift per checked step (max abs):", {k: f"{v:.2e}" for k, v in sorted(res.per_step.items())})
    # the final cache in full: 131 072 rows x 8 KV heads, keys against the oracle's rotation, values verbatim
    bits = assert_chain_cache_bits(cache, w, chunks, seed=22, what="config 3 cache")
    assert bits.elements == 131072 * 8 * 128
    print(f"config3 cache: {bits.differing} of {bits.elements} key elements differ, max {bits.max_ulp} ulp")


@pytest.mark.parametrize("C", [128, 512, 2048, 8192])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_config4_chunk_and_precision_sweep_64k(C, dtype):
    w = workloads.sweep(C, dtype)
    steps = _steps(w.n_steps, np.random.default_rng(C))
    res, cache, _, _ = run_chain(w, [C] * w.n_steps, seed=23, check_steps=steps, rows_per_step=ROWS_EXTRA)
    assert len(cache) == 65536
    assert_within(res, dtype, f"config 4 C={C} {dtype}")
    print(f"config4 C={C} {dtype}: max {res.max_abs:.2e} mean {res.mean_abs:.2e} rel_rms {res.rel_rms:.2e}")


def test_config5_layer_stack_reduced():
    """Config 5's structure (independent sequences x layers, each its own cache, all layers' steps
    issued per chunk on one stream, one shared workspace) at a size the oracle can follow."""
    w = workloads.FULL_STACK.with_(name="full_stack_reduced", tokens=4096, n_sequences=2, n_layers=3)
    C = w.chunk
    cfg = binding.make_config(w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, w.tokens, C, rope_base=w.rope_base)
    ws = torch.empty(binding.workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    caches = {(s, l): binding.Cache(cfg, workspace=ws) for s in range(w.n_sequences) for l in range(w.n_layers)}
    oracles = {key: oracle.OracleCache(w.n_q_heads, w.n_kv_heads, w.head_dim, w.tokens, rope_base=w.rope_base)
               for key in [(0, 0), (1, 2)]}
    worst = 0.0
    for t in range(w.n_steps):
        outs = {}
        for (s, l), c in caches.items():
            q, k, v = workloads.chunk_inputs(w, 24, t, sequence=s, layer=l, device="cuda")
            outs[(s, l)] = (c.fold_step(q, k, v), q, k, v)
        for key, oc in oracles.items():
            out, q, k, v = outs[key]
            rows = [0, C // 2, C - 1]
            ref = oc.fold_step(to_f64(q), to_f64(k), to_f64(v), rows=rows)
            worst = max(worst, float(np.abs(to_f64(out[rows]) - ref).max()))
    assert all(len(c) == w.tokens for c in caches.values())
    assert worst <= TOL["bf16"][0]


@pytest.mark.parametrize("batched", [False, True], ids=["per_cache_steps", "one_batch_step_per_chunk"])
def test_config5_full_stack_64_gib_sampled_pairs(batched):
    """Config 5 at full size: 4 sequences x 32 layers, one 512 MiB bf16 cache each (64 GiB), 131 072
    tokens per sequence in chunks of 1024, every chunk's 128 fold steps issued on one stream with one
    shared workspace - or, batched, as one step of a batch over 128 paged caches of one 64 GiB pool.
    Each (sequence, layer) draws one chunk of inputs from its own seed and feeds it at every chunk
    (the positions and the prefix still change), as the benchmark does; the oracle follows two
    (sequence, layer) pairs and checks sampled rows at sampled chunks."""
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < 80 * 2 ** 30:
        pytest.skip("needs 80 GiB of free device memory")
    w = workloads.FULL_STACK
    C, T, N = w.chunk, w.tokens, w.n_steps
    cfg = binding.make_config(w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, T, C, rope_base=w.rope_base)
    ws = torch.empty(binding.workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    keys = [(s, l) for s in range(w.n_sequences) for l in range(w.n_layers)]
    inputs = {key: workloads.chunk_inputs(w, 25, 0, sequence=key[0], layer=key[1], device="cuda") for key in keys}
    watched = [(0, 0), (3, 17)]
    oracles = {key: oracle.OracleCache(w.n_q_heads, w.n_kv_heads, w.head_dim, T, rope_base=w.rope_base) for key in watched}
    host_in = {key: tuple(to_f64(x) for x in inputs[key]) for key in watched}
    check_chunks = {0, 1, N // 2, N - 1}
    rows = [0, C // 2 - 1, C - 1]
    if batched:
        per = T // 128
        deck = torch.randperm(len(keys) * per, generator=torch.Generator().manual_seed(25)).to(torch.int32)
        tables = deck.view(len(keys), per).cuda()
        pool = torch.empty(binding.paged_pool_bytes(cfg, len(keys) * per), dtype=torch.uint8, device="cuda")
        caches = {key: binding.PagedCache(cfg, pool, len(keys) * per, tables[i], workspace=ws) for i, key in enumerate(keys)}
        batch = binding.Batch([caches[key] for key in keys])
        bq, bk, bv = (torch.stack([inputs[key][j] for key in keys]).contiguous() for j in range(3))
        bout = torch.empty_like(bq)
        outs = {key: bout[keys.index(key)] for key in watched}
    else:
        caches = {key: binding.Cache(cfg, workspace=ws) for key in keys}
        outs = {key: torch.empty_like(inputs[key][0]) for key in watched}
        scratch = torch.empty_like(inputs[keys[0]][0])
    worst, err_sq, ref_sq = 0.0, 0.0, 0.0
    bits = {key: CacheBits() for key in watched + [keys[0], keys[-1]]}       # the two watched pairs, first and last
    for t in range(N):
        if batched:
            batch.fold_step(bq, bk, bv, out=bout)
        else:
            for key in keys:
                q, k, v = inputs[key]
                caches[key].fold_step(q, k, v, out=outs[key] if key in outs else scratch)
        # the rows this chunk appended to the watched caches, every element (chunk t starts at row t * C)
        for key, cb in bits.items():
            _, k, v = inputs[key]
            cb.add(caches[key], w, k, v, t * C, t * C, table=tables[keys.index(key)] if batched else None)
        for key in watched:
            q, k, v = host_in[key]
            if t in check_chunks:
                ref = oracles[key].fold_step(q, k, v, rows=rows)
                got = to_f64(outs[key][rows])
                worst = max(worst, float(np.abs(got - ref).max()))
                err_sq += float(((got - ref) ** 2).sum())
                ref_sq += float((ref ** 2).sum())
            else:
                oracles[key].fold_step(q, k, v, rows=[])
    torch.cuda.synchronize()
    assert all(len(c) == T for c in caches.values())
    assert all(c.status() == binding.KVF_OK for c in caches.values())
    if batched:
        assert batch.status_word() == 0 and batch.launch_count() == 2 * N     # rotate+append and attention, no combine
    assert worst <= TOL["bf16"][0], worst
    assert (err_sq / ref_sq) ** 0.5 <= 2e-2
    for key, cb in bits.items():
        cb.check(f"config 5 cache of sequence {key[0]}, layer {key[1]}")
        assert cb.elements == T * w.n_kv_heads * w.head_dim
    print(f"config5 full size: max abs {worst:.2e}, rel rms {(err_sq / ref_sq) ** 0.5:.2e}")

"""Sink + window mask (kvf_cache_set_window) against the oracle's sink + window variant."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_12471_b200 import binding, workloads
from tests.chain import TOL, to_f64

pytestmark = pytest.mark.gpu

LLAMA = workloads.Workload("window_llama_bf16", 32, 8, 128, "bf16", 256, 1024, 500000.0)


def run(w, chunks, n_sink, window, seed, cache=None, splits=0, rows_of=None, flags=0):
    total = sum(chunks)
    if cache is None:
        cache = binding.cache_for(w, capacity=total, max_chunk=max(chunks), flags=flags)
    cache.set_window(n_sink, window)
    if splits:
        cache.set_splits(splits)
    oc = oracle.OracleCache(w.n_q_heads, w.n_kv_heads, w.head_dim, total, rope_base=w.rope_base)
    oc.set_window(n_sink, window)
    worst, worst_lse, outs = 0.0, 0.0, []
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(w, seed, t, device="cuda", n_tokens=n)
        lse = torch.empty((n, w.n_q_heads), dtype=torch.float32, device="cuda")
        out = cache.fold_step(q, k, v, lse=lse)
        outs.append(out)
        rows = list(range(n)) if rows_of is None else rows_of(n)
        ref, ref_lse, _ = oc.fold_step(to_f64(q), to_f64(k), to_f64(v), rows=rows, want_stats=True)
        worst = max(worst, float(np.abs(to_f64(out[rows]) - ref).max()))
        worst_lse = max(worst_lse, float(np.abs(to_f64(lse[rows]) - ref_lse).max()))
    torch.cuda.synchronize()
    assert cache.status() == binding.KVF_OK, hex(cache.status_word())
    return worst, worst_lse, outs, cache


def some_rows(n):
    return sorted({0, 1, n // 2, n - 2, n - 1} & set(range(n)))


def test_tiny_fp32_window_matches_oracle_everywhere():
    """CUDA-core path, d = 64: every row of every step; window edges inside tiles (100 is no multiple of 64)."""
    w = workloads.TINY
    worst, worst_lse, _, _ = run(w, [w.chunk] * w.n_steps, n_sink=4, window=100, seed=71)
    assert worst <= TOL["f32"][0] and worst_lse <= 1e-5, (worst, worst_lse)


@pytest.mark.parametrize("flags", [0, binding.KVF_FORCE_SIMT], ids=["tensor_cores", "cuda_cores"])
def test_llama_fp32_window_with_forced_splits(flags):
    w = LLAMA.with_(name="window_llama_f32", dtype="f32")
    worst, worst_lse, _, _ = run(w, [256, 256, 100, 256, 1, 256, 256], n_sink=4, window=300, seed=72, splits=3,
                                 rows_of=some_rows, flags=flags)
    assert worst <= TOL["f32"][0] and worst_lse <= 1e-5, (worst, worst_lse)


def test_llama_fp32_paper_window_on_the_tensor_cores():
    """4 sinks + 1020 recent on an fp32 cache: the sink tile, skipped tiles, a window that starts inside a
    64-key step, ragged and single-token steps behind."""
    w = LLAMA.with_(name="window_llama_f32_paper", dtype="f32")
    chunks = [256] * 8 + [100, 1, 16, 300, 1, 256]
    worst, worst_lse, _, cache = run(w, chunks, n_sink=4, window=1020, seed=75, rows_of=some_rows)
    assert cache.plan(256, 2048)[0] == 1
    assert worst <= TOL["f32"][0] and worst_lse <= 1e-5, (worst, worst_lse)


def test_llama_bf16_paper_window_4_sinks_1020_recent():
    """Tensor-core path at the published configuration (4 + 1020) with C = 256 and ragged steps behind:
    the sink tile, skipped tiles, a window that starts inside a tile, decode-shaped steps."""
    chunks = [256] * 12 + [100, 1, 16, 300, 1, 256]
    worst, worst_lse, _, cache = run(LLAMA, chunks, n_sink=4, window=1020, seed=73, rows_of=some_rows)
    assert worst <= TOL["bf16"][0] and worst_lse <= 2e-2, (worst, worst_lse)
    # the attention kernel walks the sink tile plus the window's tiles, whatever the prefix
    plan_far = cache.plan(256, 3072)
    cache.set_window(0, 0)
    plan_full = cache.plan(256, 3072)
    assert plan_far[2] <= plan_full[2]


def test_window_reaching_back_to_the_start_is_the_plain_fold_bit_for_bit():
    chunks = [256, 256, 77, 256]
    _, _, wide, _ = run(LLAMA, chunks, n_sink=4, window=10 ** 6, seed=74, rows_of=some_rows)
    _, _, plain, _ = run(LLAMA, chunks, n_sink=0, window=0, seed=74, rows_of=some_rows)
    for a, b in zip(wide, plain):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_paged_cache_never_reads_pages_outside_sinks_and_window():
    """Pages whose rows are all hidden are poisoned with NaN as soon as they fall out of the window;
    the outputs stay bit-identical to an unpoisoned contiguous cache under the same mask."""
    chunks = [256] * 10 + [1, 1, 130, 256]
    total = sum(chunks)
    n_sink, window = 4, 500
    cfg = binding.make_config(32, 8, 128, "bf16", total, 256, rope_base=LLAMA.rope_base)
    n_table = (total + 127) // 128
    perm = torch.randperm(n_table + 2, generator=torch.Generator().manual_seed(9))[:n_table].to(torch.int32)
    pool = torch.empty(binding.paged_pool_bytes(cfg, n_table + 2), dtype=torch.uint8, device="cuda")
    pool.zero_()
    paged = binding.PagedCache(cfg, pool, n_table + 2, perm.cuda())
    flat = binding.Cache(cfg)
    paged.set_window(n_sink, window)
    flat.set_window(n_sink, window)
    pages = pool.view(torch.int16).view(n_table + 2, -1)
    for t, n in enumerate(chunks):
        P = len(paged)
        # tiles wholly before the window, except the sink tile, can no longer be seen by any later chunk
        for tile in range(1, max(0, (P - window)) // 128):
            pages[int(perm[tile])].fill_(0x7FC0)
        q, k, v = workloads.chunk_inputs(LLAMA, 75, t, device="cuda", n_tokens=n)
        got = paged.fold_step(q, k, v)
        want = flat.fold_step(q, k, v)
        assert torch.equal(got.view(torch.int16), want.view(torch.int16)), f"step {t}"
        assert not torch.isnan(got.float()).any()
    torch.cuda.synchronize()
    assert paged.status() == binding.KVF_OK


def test_batch_under_a_window():
    from tests.test_batch_gpu import batch_inputs, make_members, W
    chunks = [256] * 7 + [16, 1]
    B, total = 3, sum(chunks)
    cfg, pool, tables, caches = make_members(B, total, 256, seed=21, fill=0)
    for c in caches:
        c.set_window(4, 600)
    batch = binding.Batch(caches)
    ocs = [oracle.OracleCache(W.n_q_heads, W.n_kv_heads, W.head_dim, total, rope_base=W.rope_base) for _ in range(B)]
    worst = 0.0
    for t, n in enumerate(chunks):
        q, k, v = batch_inputs(B, n, 76, t)
        out = batch.fold_step(q, k, v)
        rows = some_rows(n)
        for i in range(B):
            ocs[i].set_window(4, 600)
            ref = ocs[i].fold_step(to_f64(q[i]), to_f64(k[i]), to_f64(v[i]), rows=rows)
            worst = max(worst, float(np.abs(to_f64(out[i][rows]) - ref).max()))
    torch.cuda.synchronize()
    assert batch.status_word() == 0 and worst <= TOL["bf16"][0], worst
    caches[1].set_window(0, 0)
    q, k, v = batch_inputs(B, 1, 76, 99)
    with pytest.raises(binding.KvfError) as e:
        batch.fold_step(q, k, v)                           # members under different masks
    assert e.value.code == binding.KVF_ERR_INVALID_ARG


def test_set_window_validates():
    cache = binding.cache_for(LLAMA, capacity=1024, max_chunk=256)
    lib = binding.load()
    assert lib.kvf_cache_set_window(cache._h, -1, 10) == binding.KVF_ERR_INVALID_ARG
    assert lib.kvf_cache_set_window(cache._h, 4, 0) == binding.KVF_ERR_INVALID_ARG
    assert lib.kvf_cache_set_window(cache._h, 65, 10) == binding.KVF_ERR_UNSUPPORTED
    assert lib.kvf_cache_set_window(cache._h, 64, 1) == binding.KVF_OK
    assert lib.kvf_cache_set_window(None, 0, 0) == binding.KVF_ERR_INVALID_ARG

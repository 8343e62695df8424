"""kvf_cache_set_len: one folded haystack, several questions (the paper's multi-needle protocol queries
each key separately on the same context), and resuming from restored storage.

The oracle has no counterpart of the call: every question is checked against a FRESH oracle chain
that folds the haystack again and then that question, which is what the rolled-back cache must equal.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_12471_b200 import binding, workloads
from tests.chain import TOL, to_f64

pytestmark = pytest.mark.gpu

LLAMA = workloads.Workload("set_len_llama_bf16", 32, 8, 128, "bf16", 256, 2048, 500000.0)
HAYSTACK = [256, 256, 200]            # ends inside a 128-row key tile
QUESTION = [24, 1, 1, 1]              # a question chunk, then tokens decoded one at a time


def make_cache(kind, w, total, max_chunk):
    if kind in ("bf16", "f32"):
        return binding.cache_for(w, capacity=total, max_chunk=max_chunk)
    if kind in ("int8", "int4"):
        cfg = binding.make_config(w.n_q_heads, w.n_kv_heads, w.head_dim, "bf16", total, max_chunk, rope_base=w.rope_base,
                                  flags=binding.KVF_CACHE_INT4 if kind == "int4" else binding.KVF_CACHE_INT8)
        return binding.Cache(cfg)
    assert kind == "paged"
    cfg = binding.make_config(w.n_q_heads, w.n_kv_heads, w.head_dim, "bf16", total, max_chunk, rope_base=w.rope_base)
    n_pages = (total + 127) // 128
    pool = torch.empty(binding.paged_pool_bytes(cfg, n_pages + 3), dtype=torch.uint8, device="cuda")
    table = torch.arange(n_pages + 2, 2, -1, dtype=torch.int32, device="cuda")      # pages in reverse order
    return binding.PagedCache(cfg, pool, n_pages + 3, table)


def oracle_for(kind, w, total):
    oc = oracle.OracleCache(w.n_q_heads, w.n_kv_heads, w.head_dim, total, rope_base=w.rope_base)
    if kind in ("int8", "int4"):
        oc.set_quant(4 if kind == "int4" else 8)
    return oc


@pytest.mark.parametrize("kind", ["bf16", "f32", "int8", "int4", "paged"])
def test_several_questions_on_one_folded_haystack(kind):
    w = LLAMA.with_(name="set_len_" + kind, dtype="f32" if kind == "f32" else "bf16")
    tol = TOL["f32" if kind == "f32" else "bf16"][0]
    hay = sum(HAYSTACK)
    total = hay + sum(QUESTION)
    cache = make_cache(kind, w, total, max(HAYSTACK))
    for t, n in enumerate(HAYSTACK):
        q, k, v = workloads.chunk_inputs(w, 500, t, device="cuda", n_tokens=n)
        cache.fold_step(q, k, v)
    assert len(cache) == hay
    for key in range(3):
        # the reference: the haystack folded again from nothing, then this key's question
        oc = oracle_for(kind, w, total)
        for t, n in enumerate(HAYSTACK):
            q, k, v = workloads.chunk_inputs(w, 500, t, device="cuda", n_tokens=n)
            oc.fold_step(to_f64(q), to_f64(k), to_f64(v), rows=[])
        worst = 0.0
        for t, n in enumerate(QUESTION):
            q, k, v = workloads.chunk_inputs(w, 600 + key, t, device="cuda", n_tokens=n)
            lse = torch.empty((n, w.n_q_heads), dtype=torch.float32, device="cuda")
            out = cache.fold_step(q, k, v, lse=lse)
            ref, ref_lse, _ = oc.fold_step(to_f64(q), to_f64(k), to_f64(v), want_stats=True)
            worst = max(worst, float(np.abs(to_f64(out) - ref).max()))
            assert float(np.abs(to_f64(lse) - ref_lse).max()) <= (1e-5 if kind == "f32" else 2e-2)
            assert len(cache) == len(oc)
        assert worst <= tol, (key, worst)
        cache.set_len(hay)
        assert len(cache) == hay
    torch.cuda.synchronize()
    assert cache.status() == binding.KVF_OK, hex(cache.status_word())


def test_rolling_back_leaves_the_bits_of_a_cache_that_never_went_further():
    """Rows below the new length are untouched, rows appended after the roll-back are those of a cache
    that folded only the kept chunks, and so are the outputs, bit for bit."""
    w = LLAMA
    chunks = [256, 100, 30]
    extra = [40, 1]
    total = sum(chunks) + sum(extra) + 64
    a = binding.cache_for(w, capacity=total, max_chunk=256)
    b = binding.cache_for(w, capacity=total, max_chunk=256)
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(w, 510, t, device="cuda", n_tokens=n)
        a.fold_step(q, k, v)
        b.fold_step(q, k, v)
    keep = sum(chunks)
    before_k, before_v = a.k_plane()[:, :keep].clone(), a.v_plane()[:, :keep].clone()
    for t, n in enumerate(extra):                      # a goes further, then comes back
        q, k, v = workloads.chunk_inputs(w, 511, t, device="cuda", n_tokens=n)
        a.fold_step(q, k, v)
    a.set_len(keep)
    assert torch.equal(a.k_plane()[:, :keep], before_k) and torch.equal(a.v_plane()[:, :keep], before_v)
    for t, n in enumerate([64, 1, 7]):
        q, k, v = workloads.chunk_inputs(w, 512, t, device="cuda", n_tokens=n)
        out_a = a.fold_step(q, k, v)
        out_b = b.fold_step(q, k, v)
        assert torch.equal(out_a.view(torch.int16), out_b.view(torch.int16)), t
    n_rows = len(a)
    assert n_rows == len(b)
    assert torch.equal(a.k_plane()[:, :n_rows], b.k_plane()[:, :n_rows])
    assert torch.equal(a.v_plane()[:, :n_rows], b.v_plane()[:, :n_rows])
    torch.cuda.synchronize()
    assert a.status() == binding.KVF_OK and b.status() == binding.KVF_OK


def test_resuming_from_a_copy_of_the_storage():
    """The planes and the length are the whole state of the fold: a second cache given a byte copy of the
    first one's storage and its length continues with the same output bits."""
    w = LLAMA
    chunks = [256, 256, 77]
    total = sum(chunks) + 300
    a = binding.cache_for(w, capacity=total, max_chunk=256)
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(w, 520, t, device="cuda", n_tokens=n)
        a.fold_step(q, k, v)
    b = binding.cache_for(w, capacity=total, max_chunk=256)
    torch.cuda.synchronize()
    b.storage.copy_(a.storage)
    b.set_len(len(a))
    assert len(b) == sum(chunks)
    for t, n in enumerate([200, 1, 33]):
        q, k, v = workloads.chunk_inputs(w, 521, t, device="cuda", n_tokens=n)
        lse_a = torch.empty((n, w.n_q_heads), dtype=torch.float32, device="cuda")
        lse_b = torch.empty_like(lse_a)
        out_a = a.fold_step(q, k, v, lse=lse_a)
        out_b = b.fold_step(q, k, v, lse=lse_b)
        assert torch.equal(out_a.view(torch.int16), out_b.view(torch.int16)), t
        assert torch.equal(lse_a, lse_b), t
    torch.cuda.synchronize()
    assert a.status() == binding.KVF_OK and b.status() == binding.KVF_OK


def test_lengths_outside_the_capacity_are_refused_and_change_nothing():
    w = workloads.TINY
    cache = binding.cache_for(w, capacity=256, max_chunk=64)
    q, k, v = workloads.chunk_inputs(w, 530, 0, device="cuda", n_tokens=64)
    cache.fold_step(q, k, v)
    lib = binding.load()
    assert lib.kvf_cache_set_len(cache._h, -1) == binding.KVF_ERR_CAPACITY
    assert lib.kvf_cache_set_len(cache._h, 257) == binding.KVF_ERR_CAPACITY
    assert len(cache) == 64
    assert lib.kvf_cache_set_len(cache._h, 256) == binding.KVF_OK and len(cache) == 256
    assert lib.kvf_cache_set_len(cache._h, 0) == binding.KVF_OK and len(cache) == 0
    assert lib.kvf_cache_set_len(None, 0) == binding.KVF_ERR_INVALID_ARG

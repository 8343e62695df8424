"""One sequence whose cache rows are dealt to several caches chunk by chunk (the row-range split of
multi.py): the cache that takes a chunk folds it, the others answer the same queries over the rows
they hold (kvf_attend), kvf_merge_partials puts the parts together.  The "ranks" here are caches on
one GPU, run one after the other; the merged result must be the oracle's plain fold of the sequence."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_12471_b200 import binding, multi, workloads
from tests.chain import TOL, to_f64

pytestmark = pytest.mark.gpu

LLAMA = workloads.Workload("row_range_llama_bf16", 32, 8, 128, "bf16", 256, 4096, 500000.0)


def make_cache(kind, w, total, max_chunk, flags=0):
    if kind in ("int8", "int4"):
        flags |= binding.KVF_CACHE_INT4 if kind == "int4" else binding.KVF_CACHE_INT8
        cfg = binding.make_config(w.n_q_heads, w.n_kv_heads, w.head_dim, "bf16", total, max_chunk, rope_base=w.rope_base,
                                  flags=flags)
        return binding.Cache(cfg)
    if kind == "paged":
        cfg = binding.make_config(w.n_q_heads, w.n_kv_heads, w.head_dim, "bf16", total, max_chunk, rope_base=w.rope_base,
                                  flags=flags)
        n_pages = (total + 127) // 128
        pool = torch.empty(binding.paged_pool_bytes(cfg, n_pages), dtype=torch.uint8, device="cuda")
        table = torch.arange(n_pages - 1, -1, -1, dtype=torch.int32, device="cuda")      # pages in reverse order
        return binding.PagedCache(cfg, pool, n_pages, table)
    return binding.cache_for(w, capacity=total, max_chunk=max_chunk, flags=flags)


def run_split(w, kind, chunks, world, seed, flags=0):
    total = sum(chunks)
    caches = [make_cache(kind, w, total, max(chunks), flags) for _ in range(world)]
    oc = oracle.OracleCache(w.n_q_heads, w.n_kv_heads, w.head_dim, total, rope_base=w.rope_base)
    if kind in ("int8", "int4"):
        oc.set_quant(4 if kind == "int4" else 8)
    worst, worst_lse, pos = 0.0, 0.0, 0
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(w, seed, t, device="cuda", n_tokens=n)
        outs, lses = [], []
        for r in range(world):
            lse = torch.empty((n, w.n_q_heads), dtype=torch.float32, device="cuda")
            if multi.chunk_owner(t, world) == r:
                out = caches[r].fold_step(q, k, v, pos0=pos, lse=lse)
            elif len(caches[r]) > 0:
                out = caches[r].attend(q, pos0=pos, lse=lse)
            else:
                out = torch.zeros((n, w.n_q_heads, w.head_dim), dtype=caches[r].out_dtype, device="cuda")
                lse.fill_(float("-inf"))
            outs.append(out)
            lses.append(lse)
        out, lse = binding.merge_partials(torch.stack(outs), torch.stack(lses))
        rows = sorted({0, 1, n // 2, n - 1} & set(range(n)))
        ref, ref_lse, _ = oc.fold_step(to_f64(q), to_f64(k), to_f64(v), pos0=pos, rows=rows, want_stats=True)
        worst = max(worst, float(np.abs(to_f64(out[rows]) - ref).max()))
        worst_lse = max(worst_lse, float(np.abs(to_f64(lse[rows]) - ref_lse).max()))
        pos += n
    torch.cuda.synchronize()
    for c in caches:
        assert c.status() == binding.KVF_OK, hex(c.status_word())
    assert sum(len(c) for c in caches) == total
    return worst, worst_lse


# long chunks, ragged ones, decode-shaped steps (the decode kernel), a question-sized chunk (two streams)
CHUNKS = [256, 256, 100, 256, 1, 1, 2, 33, 256, 512, 7, 1]


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("kind", ["bf16", "f32", "int8", "int4", "paged"])
def test_rows_dealt_to_several_caches_give_the_plain_fold(kind, world):
    w = LLAMA.with_(name=f"row_range_{kind}", dtype="f32" if kind == "f32" else "bf16")
    worst, worst_lse = run_split(w, kind, CHUNKS, world, seed=41)
    assert worst <= TOL["f32" if kind == "f32" else "bf16"][0], worst
    assert worst_lse <= (1e-5 if kind == "f32" else 2e-2), worst_lse


def test_split_with_fp32_parts_and_groups_of_seven():
    """Qwen2.5-7B's 28 / 4 heads, parts exchanged in fp32 (KVF_OUT_F32): no second rounding in the merge."""
    w = workloads.Workload("row_range_qwen", 28, 4, 128, "bf16", 256, 4096, 500000.0)
    worst, worst_lse = run_split(w, "bf16", CHUNKS, 2, seed=42, flags=binding.KVF_OUT_F32)
    assert worst <= TOL["bf16"][0] and worst_lse <= 2e-2, (worst, worst_lse)


def test_tiny_fp32_split_on_the_cuda_core_path():
    w = workloads.TINY
    worst, worst_lse = run_split(w, "f32", [64, 64, 10, 1, 64, 3, 64], 2, seed=43)
    assert worst <= TOL["f32"][0] and worst_lse <= 1e-5, (worst, worst_lse)


def test_attend_changes_neither_length_nor_rows_and_refuses_what_it_cannot_do():
    w = LLAMA
    cache = binding.cache_for(w, capacity=1024, max_chunk=256)
    q, k, v = workloads.chunk_inputs(w, 44, 0, device="cuda", n_tokens=200)
    lib = binding.load()
    out = torch.empty_like(q)
    assert lib.kvf_attend(cache._h, q.data_ptr(), 200, 0, out.data_ptr(), None, None) == binding.KVF_ERR_INVALID_ARG   # empty
    cache.fold_step(q, k, v)
    planes = cache.storage.clone()
    a = cache.attend(q[:5].contiguous(), pos0=200)
    b = cache.attend(q[:5].contiguous(), pos0=200)
    torch.cuda.synchronize()
    assert len(cache) == 200 and torch.equal(cache.storage, planes)
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    assert lib.kvf_attend(cache._h, q.data_ptr(), 0, 0, out.data_ptr(), None, None) == binding.KVF_ERR_INVALID_ARG
    assert lib.kvf_attend(cache._h, q.data_ptr(), 257, 0, out.data_ptr(), None, None) == binding.KVF_ERR_INVALID_ARG
    assert lib.kvf_attend(None, q.data_ptr(), 1, 0, out.data_ptr(), None, None) == binding.KVF_ERR_INVALID_ARG
    cache.set_window(4, 100)
    assert lib.kvf_attend(cache._h, q.data_ptr(), 5, 200, out.data_ptr(), None, None) == binding.KVF_ERR_UNSUPPORTED
    assert cache.status() == binding.KVF_OK

"""Group sizes that are no power of two: the attention shapes of the other models the paper runs
(Qwen2.5-7B: 28 query / 4 KV heads, groups of 7; Qwen2.5-1.5B: 12 / 2, groups of 6; OLMoE: 16 / 16).
The tensor-core kernels lay such a group out as the next power of two; the padding rows are
computed and never written, so every output is compared with the oracle and the memory around
the outputs is checked to be untouched."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_12471_b200 import binding, workloads
from tests.chain import TOL, assert_chain_cache_bits, assert_within, run_chain, to_f64

pytestmark = pytest.mark.gpu

SHAPES = {"qwen7b_28_4": (28, 4), "qwen1p5b_12_2": (12, 2), "three_24_8": (24, 8), "olmoe_16_16": (16, 16),
          "five_5_1": (5, 1)}
# long chunks, a ragged one, decode-shaped steps (one and two tokens), a question-sized chunk
CHUNKS = [256, 100, 1, 2, 33, 256, 7, 1]


def shape(name, dtype):
    h, hkv = SHAPES[name]
    return workloads.Workload(f"groups_{name}_{dtype}", h, hkv, 128, dtype, 256, 1024, 500000.0)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("name", list(SHAPES))
def test_fold_matches_the_oracle_for_any_group_size(name, dtype):
    w = shape(name, dtype)
    res, cache, _, _ = run_chain(w, CHUNKS, seed=31)
    assert len(cache) == sum(CHUNKS)
    assert cache.plan(256)[0] == 1, "the tensor-core path serves this shape"
    assert_within(res, dtype, w.name)
    assert res.lse_max_abs <= (1e-5 if dtype == "f32" else 2e-2), res.lse_max_abs
    if dtype == "bf16":
        assert_chain_cache_bits(cache, w, CHUNKS, 31, what=w.name)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_groups_of_seven_with_the_key_range_cut_in_pieces(dtype):
    """Forced splits: every step leaves partial results in the padded row layout and the merge reads them."""
    w = shape("qwen7b_28_4", dtype)
    chunks = [512, 256, 40, 2, 1, 256]
    for splits in (2, 5):
        res, cache, _, _ = run_chain(w, chunks, seed=32, splits=splits, check_steps=[1, 2, 3, 4, 5], rows_per_step=4)
        assert cache.plan(256)[1] == splits
        assert_within(res, dtype, f"{w.name} splits={splits}")


def test_padding_rows_are_never_written():
    """Outputs and log-sum-exps sit in the middle of buffers filled with a pattern: nothing around them changes."""
    w = shape("qwen7b_28_4", "bf16")
    cache = binding.cache_for(w, capacity=1024, max_chunk=256)
    H, d = w.n_q_heads, w.head_dim
    for t, n in enumerate([256, 19, 2, 130]):
        q, k, v = workloads.chunk_inputs(w, 33, t, device="cuda", n_tokens=n)
        guard = 4 * H * d
        buf = torch.full((2 * guard + n * H * d,), -7.0, dtype=torch.bfloat16, device="cuda")
        lbuf = torch.full((2 * H + n * H,), -7.0, dtype=torch.float32, device="cuda")
        out = buf[guard:guard + n * H * d].view(n, H, d)
        lse = lbuf[H:H + n * H].view(n, H)
        cache.fold_step(q, k, v, out=out, lse=lse)
        torch.cuda.synchronize()
        assert bool((buf[:guard] == -7.0).all()) and bool((buf[guard + n * H * d:] == -7.0).all()), t
        assert bool((lbuf[:H] == -7.0).all()) and bool((lbuf[H + n * H:] == -7.0).all()), t
        assert bool(torch.isfinite(out.float()).all()) and bool(torch.isfinite(lse).all())
    assert cache.status() == binding.KVF_OK


@pytest.mark.parametrize("bits", [8, 4], ids=["int8", "int4"])
def test_quantised_cache_with_groups_of_seven(bits):
    w = shape("qwen7b_28_4", "bf16")
    chunks = [512, 256, 100, 1, 2, 30, 512]          # 512 tokens x 8 padded rows: the paired long-chunk kernel too
    total = sum(chunks)
    cfg = binding.make_config(w.n_q_heads, w.n_kv_heads, w.head_dim, "bf16", total, max(chunks), rope_base=w.rope_base,
                              flags=binding.KVF_CACHE_INT4 if bits == 4 else binding.KVF_CACHE_INT8)
    cache = binding.Cache(cfg)
    oc = oracle.OracleCache(w.n_q_heads, w.n_kv_heads, w.head_dim, total, rope_base=w.rope_base)
    oc.set_quant(bits)
    worst = 0.0
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(w, 34, t, device="cuda", n_tokens=n)
        out = cache.fold_step(q, k, v)
        rows = sorted({0, 1, n // 2, n - 1} & set(range(n)))
        ref = oc.fold_step(to_f64(q), to_f64(k), to_f64(v), rows=rows)
        worst = max(worst, float(np.abs(to_f64(out[rows]) - ref).max()))
    torch.cuda.synchronize()
    assert cache.status() == binding.KVF_OK, hex(cache.status_word())
    assert worst <= TOL["bf16"][0], worst


def test_batch_of_paged_caches_with_groups_of_seven():
    """Three sequences of different length decoded and extended together (ragged batch) on pages."""
    w = shape("qwen7b_28_4", "bf16")
    B, cap = 3, 1024
    cfg = binding.make_config(w.n_q_heads, w.n_kv_heads, w.head_dim, "bf16", cap, 256, rope_base=w.rope_base)
    per = cap // 128
    pool = torch.empty(binding.paged_pool_bytes(cfg, B * per), dtype=torch.uint8, device="cuda")
    tables = torch.randperm(B * per, generator=torch.Generator().manual_seed(5)).to(torch.int32).view(B, per).cuda()
    caches = [binding.PagedCache(cfg, pool, B * per, tables[i]) for i in range(B)]
    ocs = [oracle.OracleCache(w.n_q_heads, w.n_kv_heads, w.head_dim, cap, rope_base=w.rope_base) for _ in range(B)]
    # different prefixes, folded per cache
    for i, pre in enumerate([256, 130, 40]):
        q, k, v = workloads.chunk_inputs(w, 35, 100 + i, device="cuda", n_tokens=pre)
        caches[i].fold_step(q, k, v)
        ocs[i].fold_step(to_f64(q), to_f64(k), to_f64(v), rows=[])
    batch = binding.Batch(caches)
    worst = 0.0
    for t, n in enumerate([2, 1, 40, 1]):
        qs, ks, vs = zip(*[workloads.chunk_inputs(w, 36 + i, t, device="cuda", n_tokens=n) for i in range(B)])
        out = batch.fold_step(torch.stack(qs), torch.stack(ks), torch.stack(vs), ragged=True)
        for i in range(B):
            ref = ocs[i].fold_step(to_f64(qs[i]), to_f64(ks[i]), to_f64(vs[i]))
            worst = max(worst, float(np.abs(to_f64(out[i]) - ref).max()))
    torch.cuda.synchronize()
    assert batch.status_word() == 0
    assert worst <= TOL["bf16"][0], worst


def test_qwen_heads_on_the_deep_chain_at_full_size():
    """28 / 4 heads through the benchmark's launch configuration (`bench.py --q-heads 28 --kv-heads 4`): 512 steps
    of 256 tokens to 131 072, sampled steps and rows against the oracle, the final cache in full."""
    w = workloads.DEEP_CHAIN.with_(name="deep_chain_qwen_28_4", n_q_heads=28, n_kv_heads=4)
    chunks = [w.chunk] * w.n_steps
    rng = np.random.default_rng(7)
    steps = sorted({0, 1, w.n_steps // 2, w.n_steps - 2, w.n_steps - 1} | {int(x) for x in rng.integers(0, w.n_steps, size=4)})
    res, cache, _, _ = run_chain(w, chunks, seed=37, check_steps=steps, rows_per_step=4)
    assert len(cache) == 131072
    assert_within(res, "bf16", "deep chain, groups of 7")
    assert res.rel_rms <= 2e-2, res.rel_rms
    bits = assert_chain_cache_bits(cache, w, chunks, seed=37, what="deep chain, groups of 7: cache")
    assert bits.elements == 131072 * 4 * 128

"""int8 cache storage (KVF_CACHE_INT8): the stored codes and scales bit for bit against the oracle's
round trip, and the fold against the oracle's quantised fold."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2605_12471_b200 import binding, workloads
from tests.chain import TOL, to_f64

pytestmark = pytest.mark.gpu

W = workloads.Workload("quant_llama_bf16", 32, 8, 128, "bf16", 256, 2048, 500000.0)


def quant_cache(total, max_chunk, flags=0, bits=8):
    cfg = binding.make_config(W.n_q_heads, W.n_kv_heads, W.head_dim, "bf16", total, max_chunk, rope_base=W.rope_base,
                              flags=flags | (binding.KVF_CACHE_INT4 if bits == 4 else binding.KVF_CACHE_INT8))
    return cfg, binding.Cache(cfg)


BITS = pytest.mark.parametrize("bits", [8, 4], ids=["int8", "int4"])


@BITS
@pytest.mark.parametrize("flags", [0, binding.KVF_ROPE_INTERLEAVED], ids=["rotate_half", "interleaved"])
def test_stored_codes_and_scales_are_the_oracles_round_trip(flags, bits):
    chunks = [256, 100, 1, 16, 300]
    total = sum(chunks)
    cfg, cache = quant_cache(total, max(chunks), flags, bits)
    assert binding.cache_storage_bytes(cfg) == 2 * W.n_kv_heads * (total * W.head_dim * bits // 8 + (total + 3) // 4 * 4 * 4)
    tab = oracle.inv_freq(W.rope_base, W.head_dim)
    t0 = 0
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(W, 101, t, device="cuda", n_tokens=n)
        cache.fold_step(q, k, v)
        rot = oracle.rope_faithful(k.float().cpu().numpy(), t0, tab, interleaved=bool(flags))       # fp32, no bf16 rounding
        kc, ks, _ = oracle.quant_rows(rot, bits)
        vc, vs, _ = oracle.quant_rows(v.float().cpu().numpy(), bits)
        got_kc = cache.k_plane()[:, t0:t0 + n].cpu().numpy().astype(np.int32)                       # [Hkv, n, d]
        got_vc = cache.v_plane()[:, t0:t0 + n].cpu().numpy().astype(np.int32)
        assert np.array_equal(got_kc, np.transpose(kc, (1, 0, 2))), f"key codes, step {t}"
        assert np.array_equal(got_vc, np.transpose(vc, (1, 0, 2))), f"value codes, step {t}"
        assert np.array_equal(cache.scales(0)[:, t0:t0 + n].cpu().numpy().view(np.uint32), ks.T.copy().view(np.uint32))
        assert np.array_equal(cache.scales(1)[:, t0:t0 + n].cpu().numpy().view(np.uint32), vs.T.copy().view(np.uint32))
        t0 += n
    torch.cuda.synchronize()
    assert cache.status() == binding.KVF_OK


@BITS
def test_quantised_fold_matches_the_quantised_oracle(bits):
    chunks = [256, 256, 100, 1, 16, 300, 256, 1]
    total = sum(chunks)
    cfg, cache = quant_cache(total, max(chunks), bits=bits)
    oc = oracle.OracleCache(W.n_q_heads, W.n_kv_heads, W.head_dim, total, rope_base=W.rope_base)
    oc.set_quant(bits)
    plain = oracle.OracleCache(W.n_q_heads, W.n_kv_heads, W.head_dim, total, rope_base=W.rope_base)
    worst, worst_lse, err_sq, ref_sq, dq_sq = 0.0, 0.0, 0.0, 0.0, 0.0
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(W, 102, t, device="cuda", n_tokens=n)
        lse = torch.empty((n, W.n_q_heads), dtype=torch.float32, device="cuda")
        out = cache.fold_step(q, k, v, lse=lse)
        rows = sorted({0, 1, n // 2, n - 1} & set(range(n)))
        ref, ref_lse, _ = oc.fold_step(to_f64(q), to_f64(k), to_f64(v), rows=rows, want_stats=True)
        unq = plain.fold_step(to_f64(q), to_f64(k), to_f64(v), rows=rows)
        got = to_f64(out[rows])
        worst = max(worst, float(np.abs(got - ref).max()))
        worst_lse = max(worst_lse, float(np.abs(to_f64(lse[rows]) - ref_lse).max()))
        err_sq += float(((got - ref) ** 2).sum())
        ref_sq += float((ref ** 2).sum())
        dq_sq += float(((ref - unq) ** 2).sum())
    torch.cuda.synchronize()
    assert cache.status() == binding.KVF_OK and len(cache) == total
    assert worst <= TOL["bf16"][0] and worst_lse <= 2e-2, (worst, worst_lse)
    # the kernel's own error is well below what the quantisation itself moves the outputs by
    assert err_sq < dq_sq, (err_sq, dq_sq)
    print(f"int{bits} cache: max abs vs quantised oracle {worst:.2e}, rel rms {np.sqrt(err_sq / ref_sq):.2e}; "
          f"quantisation moved the outputs by rel rms {np.sqrt(dq_sq / ref_sq):.2e}")


def test_quantised_storage_rejects_what_it_does_not_cover():
    lib = binding.load()
    h = ctypes.c_void_p()
    both = binding.make_config(32, 8, 128, "bf16", 1024, 256, rope_base=5e5, flags=binding.KVF_CACHE_INT8 | binding.KVF_CACHE_INT4)
    assert lib.kvf_cache_create(ctypes.byref(both), 256, 1 << 30, 256, 1 << 30, ctypes.byref(h)) == binding.KVF_ERR_INVALID_ARG
    f32 = binding.make_config(32, 8, 128, "f32", 1024, 256, rope_base=5e5, flags=binding.KVF_CACHE_INT8)
    assert binding.cache_storage_bytes(f32) == 0
    assert lib.kvf_cache_create(ctypes.byref(f32), 256, 1 << 30, 256, 1 << 30, ctypes.byref(h)) == binding.KVF_ERR_UNSUPPORTED
    d64 = binding.make_config(4, 1, 64, "bf16", 1024, 256, flags=binding.KVF_CACHE_INT8)
    assert lib.kvf_cache_create(ctypes.byref(d64), 256, 1 << 30, 256, 1 << 30, ctypes.byref(h)) == binding.KVF_ERR_UNSUPPORTED
    cfg = binding.make_config(32, 8, 128, "bf16", 1024, 256, rope_base=5e5, flags=binding.KVF_CACHE_INT8)
    buf = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")
    table = torch.zeros(8, dtype=torch.int32, device="cuda")
    ws = torch.empty(binding.workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    rc = lib.kvf_paged_cache_create(ctypes.byref(cfg), buf.data_ptr(), buf.numel(), 8, table.data_ptr(), ws.data_ptr(),
                                    ws.numel(), ctypes.byref(h))
    assert rc == binding.KVF_OK                     # quantised rows may live in pages (8 pages of 264 KiB fit 64 MiB)
    lib.kvf_cache_destroy(h)
    rc = lib.kvf_paged_cache_create(ctypes.byref(cfg), buf.data_ptr(), 8 * 270336 - 1, 8, table.data_ptr(), ws.data_ptr(),
                                    ws.numel(), ctypes.byref(h))
    assert rc == binding.KVF_ERR_CAPACITY           # a page holds 2 x 8 x 128 rows of 128 codes + 2 x 8 x 128 scales
    plain = binding.make_config(32, 8, 128, "bf16", 1024, 256, rope_base=5e5)
    assert binding.workspace_bytes(cfg) == binding.workspace_bytes(plain)          # no bf16 image of the cache anywhere


@BITS
def test_quantised_fold_decode_steps_at_depth_and_forced_splits(bits):
    """Decode-shaped steps (two streams, rings of two slots) behind a 6 144-token prefix, then the same
    cache with the key range cut three ways per KV head: sampled rows against the quantised oracle."""
    prefix, steps = 6144, [1, 1, 8, 32, 1, 256, 100]
    total = prefix + sum(steps)
    cfg, cache = quant_cache(total, 2048, bits=bits)
    oc = oracle.OracleCache(W.n_q_heads, W.n_kv_heads, W.head_dim, total, rope_base=W.rope_base)
    oc.set_quant(bits)
    worst = 0.0
    for t in range(prefix // 2048):
        q, k, v = workloads.chunk_inputs(W, 103, t, device="cuda", n_tokens=2048)
        out = cache.fold_step(q, k, v)                       # two row tiles, 32 row pairs, whole KV heads or 9 groups
        rows = [0, 1023, 2047]
        ref = oc.fold_step(to_f64(q), to_f64(k), to_f64(v), rows=rows)
        worst = max(worst, float(np.abs(to_f64(out[rows]) - ref).max()))
    for t, n in enumerate(steps):
        if t == 4:
            cache.set_splits(3)
        q, k, v = workloads.chunk_inputs(W, 104, t, device="cuda", n_tokens=n)
        out = cache.fold_step(q, k, v)
        rows = sorted({0, n // 2, n - 1})
        ref = oc.fold_step(to_f64(q), to_f64(k), to_f64(v), rows=rows)
        worst = max(worst, float(np.abs(to_f64(out[rows]) - ref).max()))
    torch.cuda.synchronize()
    assert cache.status() == binding.KVF_OK, hex(cache.status_word())
    assert worst <= TOL["bf16"][0], worst


@BITS
def test_quantised_fold_under_a_window_and_repeated_runs_give_the_same_bits(bits):
    chunks = [256] * 8 + [16, 1, 256]
    total = sum(chunks)
    runs = []
    for rep in range(2):
        cfg, cache = quant_cache(total, 256, bits=bits)
        cache.set_window(4, 700)
        oc = oracle.OracleCache(W.n_q_heads, W.n_kv_heads, W.head_dim, total, rope_base=W.rope_base)
        oc.set_quant(bits)
        oc.set_window(4, 700)
        outs, worst = [], 0.0
        for t, n in enumerate(chunks):
            q, k, v = workloads.chunk_inputs(W, 105, t, device="cuda", n_tokens=n)
            outs.append(cache.fold_step(q, k, v))               # no synchronisation between the steps
            if rep == 0:
                rows = sorted({0, n // 2, n - 1})
                ref = oc.fold_step(to_f64(q), to_f64(k), to_f64(v), rows=rows)
                worst = max(worst, float(np.abs(to_f64(outs[-1][rows]) - ref).max()))
        torch.cuda.synchronize()
        assert cache.status() == binding.KVF_OK, hex(cache.status_word())
        assert worst <= TOL["bf16"][0], worst
        runs.append(torch.cat(outs))
    assert torch.equal(runs[0].view(torch.int16), runs[1].view(torch.int16))


@BITS
def test_quantised_deep_chain_32k_sampled_steps(bits):
    """The benchmark's launch shape (C = 256, 148 CTAs, pieces that straddle KV heads) on an int8 cache,
    128 steps deep; sampled steps and rows against the quantised oracle."""
    C, N = 256, 128
    cfg, cache = quant_cache(C * N, C, bits=bits)
    oc = oracle.OracleCache(W.n_q_heads, W.n_kv_heads, W.head_dim, C * N, rope_base=W.rope_base)
    oc.set_quant(bits)
    check = {0, 1, 2, 31, 64, 126, 127}
    worst, err_sq, ref_sq = 0.0, 0.0, 0.0
    for t in range(N):
        q, k, v = workloads.chunk_inputs(W, 106, t, device="cuda", n_tokens=C)
        out = cache.fold_step(q, k, v)
        rows = [0, 100, 255] if t in check else []
        ref = oc.fold_step(to_f64(q), to_f64(k), to_f64(v), rows=rows)
        if rows:
            got = to_f64(out[rows])
            worst = max(worst, float(np.abs(got - ref).max()))
            err_sq += float(((got - ref) ** 2).sum())
            ref_sq += float((ref ** 2).sum())
    torch.cuda.synchronize()
    assert cache.status() == binding.KVF_OK, hex(cache.status_word())
    assert worst <= TOL["bf16"][0] and (err_sq / ref_sq) ** 0.5 <= 2e-2, (worst, (err_sq / ref_sq) ** 0.5)


# ------------------------------------------------------------------ quantised rows in pages, and batches of them
def quant_paged_members(n_caches, capacity, max_chunk, bits, seed):
    """n_caches paged caches with quantised storage over one pool, pages dealt from one shuffled deck."""
    cfg = binding.make_config(W.n_q_heads, W.n_kv_heads, W.head_dim, "bf16", capacity, max_chunk, rope_base=W.rope_base,
                              flags=binding.KVF_CACHE_INT4 if bits == 4 else binding.KVF_CACHE_INT8)
    per = (capacity + 127) // 128
    n_pool = n_caches * per + 2
    deck = torch.randperm(n_pool, generator=torch.Generator().manual_seed(seed))[:n_caches * per].to(torch.int32)
    tables = deck.view(n_caches, per).cuda()
    pool = torch.empty(binding.paged_pool_bytes(cfg, n_pool), dtype=torch.uint8, device="cuda")
    pool.fill_(0xFF)                                        # scale bits 0xFFFFFFFF = NaN wherever no row was written
    ws = torch.empty(binding.workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    caches = [binding.PagedCache(cfg, pool, n_pool, tables[i], workspace=ws) for i in range(n_caches)]
    return cfg, pool, tables, caches


@BITS
def test_paged_quantised_cache_holds_the_same_codes_and_gives_the_same_bits(bits):
    """Codes and scales in 128-token pages scattered over a pool: the same codes, scales and output bits as
    the contiguous quantised cache (whose codes are the oracle's), ragged and single-token steps included."""
    chunks = [256, 100, 1, 16, 300, 128, 33]
    total = sum(chunks)
    cfg, pool, tables, (paged,) = quant_paged_members(1, total, max(chunks), bits, seed=3)
    assert binding.paged_pool_bytes(cfg, 4) == 4 * (2 * 8 * 128 * (128 * bits // 8) + 2 * 8 * 128 * 4)
    _, flat = quant_cache(total, max(chunks), bits=bits)
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(W, 105, t, device="cuda", n_tokens=n)
        got = paged.fold_step(q, k, v)
        want = flat.fold_step(q, k, v)
        assert torch.equal(got.view(torch.int16), want.view(torch.int16)), f"step {t}"
    torch.cuda.synchronize()
    assert paged.status() == binding.KVF_OK and len(paged) == total
    table = tables[0].cpu()
    for kv in (0, 1):
        codes, scales = paged.page_codes(kv), paged.page_scales(kv)
        flat_codes = flat.k_plane() if kv == 0 else flat.v_plane()
        flat_scales = flat.scales(kv)
        for i in range((total + 127) // 128):
            rows = min(128, total - 128 * i)
            page = int(table[i])
            assert torch.equal(codes[page, :, :rows], flat_codes[:, 128 * i:128 * i + rows]), (kv, i)
            assert torch.equal(scales[page, :, :rows].view(torch.int32), flat_scales[:, 128 * i:128 * i + rows].contiguous().view(torch.int32)), (kv, i)


@BITS
def test_two_ctas_sharing_their_expansions_give_the_bits_of_ctas_on_their_own(bits):
    """Chunks whose row pairs come in twos (128, 256, 512, 1024 tokens) run as clusters of two CTAs, each expanding
    half of every code tile for both, at any prefix: the two walk the key tiles of the later row pair, and the
    earlier one masks what it does not see (the chunks after the 100-token one start off the tile grid).  A step
    whose members may take fewer tokens than the chunk (kvf_batch_fold_step_varlen, here a batch of one cache
    taking all of them) never does.  Wherever both cut the key range alike the outputs are the same bits; everywhere they
    agree within the tolerance, and with the oracle's quantised fold on sampled rows."""
    chunks = [256] * 5 + [100] + [256] * 4 + [512, 1024, 256, 128, 256]
    total = sum(chunks)
    _, _, _, (alone,) = quant_paged_members(1, total, max(chunks), bits, seed=11)
    _, _, _, (member,) = quant_paged_members(1, total, max(chunks), bits, seed=11)
    batch = binding.Batch([member])
    oc = oracle.OracleCache(W.n_q_heads, W.n_kv_heads, W.head_dim, total, rope_base=W.rope_base)
    oc.set_quant(bits)
    same_plan, worst, worst_oracle = 0, 0.0, 0.0
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(W, 113, t, device="cuda", n_tokens=n)
        prefix = len(alone)
        got = alone.fold_step(q, k, v)
        want = batch.fold_step_varlen(q[None].contiguous(), k[None].contiguous(), v[None].contiguous(), [n])[0]
        if alone.plan(n, prefix)[1:] == batch.plan(n, prefix)[1:]:
            same_plan += 1
            assert torch.equal(got.view(torch.int16), want.view(torch.int16)), f"step {t}"
        worst = max(worst, float((got.float() - want.float()).abs().max()))
        rows = sorted({0, 1, n // 4, n // 2 - 1, n // 2, n - 1})     # rows of both CTAs of a cluster
        ref = oc.fold_step(to_f64(q), to_f64(k), to_f64(v), rows=rows)
        worst_oracle = max(worst_oracle, float(np.abs(to_f64(got[rows]) - ref).max()))
    torch.cuda.synchronize()
    assert alone.status() == binding.KVF_OK and batch.status_word() == 0
    assert same_plan >= len(chunks) // 2, same_plan
    assert worst <= TOL["bf16"][0] and worst_oracle <= TOL["bf16"][0], (worst, worst_oracle)


@BITS
def test_batch_of_paged_quantised_caches(bits):
    """One launch over three quantised paged caches: per member the bits of its own step, outputs within
    tolerance of the oracle's quantised fold; lock-step chunks, then a ragged step."""
    chunks = [256, 100, 16, 1, 300]
    total = sum(chunks) + 64 + 32
    B = 3
    cfg, pool, tables, caches = quant_paged_members(B, total, max(chunks), bits, seed=5)
    _, pool1, _, singles = quant_paged_members(B, total, max(chunks), bits, seed=5)
    batch = binding.Batch(caches)
    ocs = [oracle.OracleCache(W.n_q_heads, W.n_kv_heads, W.head_dim, total, rope_base=W.rope_base) for _ in range(B)]
    for oc in ocs:
        oc.set_quant(bits)
    worst, worst_pair = 0.0, 0.0
    for t, n in enumerate(chunks):
        qs, ks, vs = zip(*[workloads.chunk_inputs(W, 106, t, sequence=i, device="cuda", n_tokens=n) for i in range(B)])
        q, k, v = (torch.stack(x).contiguous() for x in (qs, ks, vs))
        out = batch.fold_step(q, k, v)
        rows = sorted({0, n // 2, n - 1})
        for i in range(B):
            alone = singles[i].fold_step(q[i], k[i], v[i])
            worst_pair = max(worst_pair, float((out[i].float() - alone.float()).abs().max()))
            ref = ocs[i].fold_step(to_f64(q[i]), to_f64(k[i]), to_f64(v[i]), rows=rows)
            worst = max(worst, float(np.abs(to_f64(out[i][rows]) - ref).max()))
    # members of different length: one member gets 64 rows more on its own, then a ragged step over all three
    q1, k1, v1 = workloads.chunk_inputs(W, 107, 0, sequence=1, device="cuda", n_tokens=64)
    caches[1].fold_step(q1, k1, v1)
    singles[1].fold_step(q1, k1, v1)
    ocs[1].fold_step(to_f64(q1), to_f64(k1), to_f64(v1), rows=[])
    qs, ks, vs = zip(*[workloads.chunk_inputs(W, 108, 0, sequence=i, device="cuda", n_tokens=32) for i in range(B)])
    q, k, v = (torch.stack(x).contiguous() for x in (qs, ks, vs))
    out = batch.fold_step(q, k, v, ragged=True)
    for i in range(B):
        alone = singles[i].fold_step(q[i], k[i], v[i])
        worst_pair = max(worst_pair, float((out[i].float() - alone.float()).abs().max()))
        ref = ocs[i].fold_step(to_f64(q[i]), to_f64(k[i]), to_f64(v[i]), rows=[0, 31])
        worst = max(worst, float(np.abs(to_f64(out[i][[0, 31]]) - ref).max()))
    torch.cuda.synchronize()
    assert batch.status_word() == 0 and all(c.status() == binding.KVF_OK for c in caches)
    assert [len(c) for c in caches] == [sum(chunks) + 32, sum(chunks) + 96, sum(chunks) + 32]
    assert torch.equal(pool, pool1)                         # every code and every scale, page for page
    assert worst <= TOL["bf16"][0] and worst_pair <= TOL["bf16"][0], (worst, worst_pair)


@BITS
def test_batch_of_quantised_caches_decoding_together(bits):
    """Decode-shaped steps of a batch (at most 16 query rows per member) take the decode kernel with the cache in
    the grid: members in lock step, members of different length (one far shorter than the key ranges the longest
    one is cut into), members that take fewer tokens or sit a step out.  Per member the pool ends up bit-identical
    to folding it by itself; every row of every step against the oracle's quantised fold."""
    B = 5
    extra = [0, 40, 700, 3, 1300]                      # tokens the members fold on their own after the common prefix
    total = 2 * 2048 + max(extra) + 64
    cfg, pool, tables, caches = quant_paged_members(B, total, 2048, bits, seed=21)
    _, pool1, _, singles = quant_paged_members(B, total, 2048, bits, seed=21)
    batch = binding.Batch(caches)
    ocs = [oracle.OracleCache(W.n_q_heads, W.n_kv_heads, W.head_dim, total, rope_base=W.rope_base) for _ in range(B)]
    for oc in ocs:
        oc.set_quant(bits)

    def inputs(n, seed, t):
        qs, ks, vs = zip(*[workloads.chunk_inputs(W, seed, t, sequence=i, device="cuda", n_tokens=n) for i in range(B)])
        return tuple(torch.stack(x).contiguous() for x in (qs, ks, vs))

    worst, worst_lse, worst_pair = 0.0, 0.0, 0.0

    def check(out, lse, q, k, v, ns):
        nonlocal worst, worst_lse, worst_pair
        for i, n in enumerate(ns):
            if n == 0:
                continue
            qi, ki, vi = (x[i, :n].contiguous() for x in (q, k, v))
            alone = singles[i].fold_step(qi, ki, vi)
            worst_pair = max(worst_pair, float((out[i, :n].float() - alone.float()).abs().max()))
            rows = list(range(n)) if n <= 4 else []
            ref, ref_lse, _ = ocs[i].fold_step(to_f64(qi), to_f64(ki), to_f64(vi), rows=rows, want_stats=True)
            if rows:
                worst = max(worst, float(np.abs(to_f64(out[i, :n]) - ref).max()))
                worst_lse = max(worst_lse, float(np.abs(to_f64(lse[i, :n]) - ref_lse).max()))

    # the common prefix, in lock step (the long-chunk kernel), and two lock-step decode steps
    for t, n in enumerate([2048, 2048, 1, 4]):
        q, k, v = inputs(n, 141, t)
        lse = torch.empty((B, n, W.n_q_heads), dtype=torch.float32, device="cuda")
        if n <= 4 and torch.cuda.get_device_properties(0).multi_processor_count == 148:
            assert batch.plan(n) == (1, 3, 120, 3)             # 148 / (8 KV heads x 5 caches) = 3 ranges per head and cache
        out = batch.fold_step(q, k, v, lse=lse)
        check(out, lse, q, k, v, [n] * B)
    # members of different length
    for i, n in enumerate(extra):
        if n:
            q1, k1, v1 = workloads.chunk_inputs(W, 142, 0, sequence=i, device="cuda", n_tokens=n)
            caches[i].fold_step(q1, k1, v1)
            singles[i].fold_step(q1, k1, v1)
            ocs[i].fold_step(to_f64(q1), to_f64(k1), to_f64(v1), rows=[])
    for t, n in enumerate([1, 2, 4, 1]):
        q, k, v = inputs(n, 143, t)
        lse = torch.empty((B, n, W.n_q_heads), dtype=torch.float32, device="cuda")
        out = batch.fold_step(q, k, v, lse=lse, ragged=True)
        check(out, lse, q, k, v, [n] * B)
    # more key ranges per KV head than the members have key tiles: ranges without a tile leave empty partials
    caches[0].set_splits(48)
    q, k, v = inputs(1, 145, 0)
    lse = torch.empty((B, 1, W.n_q_heads), dtype=torch.float32, device="cuda")
    out = batch.fold_step(q, k, v, lse=lse, ragged=True)
    check(out, lse, q, k, v, [1] * B)
    caches[0].set_splits(0)
    # fewer tokens for some, none for others
    for t, (mx, ns) in enumerate([(2, [1, 0, 2, 1, 2]), (4, [4, 3, 0, 0, 1]), (1, [0, 1, 0, 1, 1])]):
        q, k, v = inputs(mx, 144, t)
        out = torch.full(q.shape, 7.0, dtype=torch.bfloat16, device="cuda")
        lse = torch.full((B, mx, W.n_q_heads), 7.0, dtype=torch.float32, device="cuda")
        batch.fold_step_varlen(q, k, v, ns, out=out, lse=lse)
        for i, n in enumerate(ns):
            assert bool((out[i, n:] == 7.0).all()) and bool((lse[i, n:] == 7.0).all())
        check(out, lse, q, k, v, ns)
    torch.cuda.synchronize()
    assert batch.status_word() == 0 and all(c.status() == binding.KVF_OK for c in caches)
    assert [len(c) for c in caches] == [len(c) for c in singles] == [len(oc) for oc in ocs]
    assert torch.equal(pool, pool1)                        # every code and every scale, page for page
    assert worst <= TOL["bf16"][0] and worst_pair <= TOL["bf16"][0] and worst_lse <= 2e-2, (worst, worst_pair, worst_lse)


@BITS
@pytest.mark.parametrize("paged", [False, True], ids=["contiguous", "paged"])
def test_decode_shaped_steps_on_a_quantised_cache_at_depth(bits, paged):
    """One to four tokens per step (at most 16 query rows) after a long prefix: the kernel that expands codes
    straight into MMA register fragments, every row of every step against the oracle's quantised fold; then
    longer chunks again (the other kernel) on the same cache, and forced range counts."""
    chunks = [2048] * 4 + [1, 1, 2, 3, 4, 1, 4] + [256, 5, 1] + [1] * 6
    total = sum(chunks)
    if paged:
        cfg, pool, tables, (cache,) = quant_paged_members(1, total, max(chunks), bits, seed=9)
    else:
        cfg, cache = quant_cache(total, max(chunks), bits=bits)
    oc = oracle.OracleCache(W.n_q_heads, W.n_kv_heads, W.head_dim, total, rope_base=W.rope_base)
    oc.set_quant(bits)
    if torch.cuda.get_device_properties(0).multi_processor_count == 148:
        assert cache.plan(1, 8192) == (1, 18, 144, 3)            # 18 key ranges per KV head, one CTA each
        assert cache.plan(4, 8192) == (1, 18, 144, 3) and cache.plan(5, 8192)[2] != 144      # 16 rows is the limit
    worst, worst_lse = 0.0, 0.0
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(W, 109, t, device="cuda", n_tokens=n)
        if t >= len(chunks) - 6:
            cache.set_splits([1, 2, 3, 7, 18, 0][t - (len(chunks) - 6)])      # one range per KV head (direct output) ... many
        lse = torch.empty((n, W.n_q_heads), dtype=torch.float32, device="cuda")
        out = cache.fold_step(q, k, v, lse=lse)
        rows = list(range(n)) if n <= 4 else []
        ref, ref_lse, _ = oc.fold_step(to_f64(q), to_f64(k), to_f64(v), rows=rows, want_stats=True)
        if rows:
            worst = max(worst, float(np.abs(to_f64(out) - ref).max()))
            worst_lse = max(worst_lse, float(np.abs(to_f64(lse) - ref_lse).max()))
    torch.cuda.synchronize()
    assert cache.status() == binding.KVF_OK and len(cache) == total
    assert worst <= TOL["bf16"][0] and worst_lse <= 2e-2, (worst, worst_lse)


def test_decode_steps_on_an_int8_cache_at_the_benchmark_prefix():
    """The decode benchmark's launch configuration: prefix 129 024 (63 steps of 2048), then steps of one, two and
    four tokens, every row of them against the oracle's quantised fold; 144 CTAs of the decode kernel."""
    chunks = [2048] * 63 + [1, 1, 2, 4, 1]
    total = sum(chunks)
    cfg, cache = quant_cache(total, 2048, bits=8)
    oc = oracle.OracleCache(W.n_q_heads, W.n_kv_heads, W.head_dim, total, rope_base=W.rope_base)
    oc.set_quant(8)
    if torch.cuda.get_device_properties(0).multi_processor_count == 148:
        assert cache.plan(1, 129024) == (1, 18, 144, 3)
    worst, worst_lse = 0.0, 0.0
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(W, 131, t, device="cuda", n_tokens=n)
        lse = torch.empty((n, W.n_q_heads), dtype=torch.float32, device="cuda")
        out = cache.fold_step(q, k, v, lse=lse)
        rows = list(range(n)) if n <= 4 else []
        ref, ref_lse, _ = oc.fold_step(to_f64(q), to_f64(k), to_f64(v), rows=rows, want_stats=True)
        if rows:
            worst = max(worst, float(np.abs(to_f64(out) - ref).max()))
            worst_lse = max(worst_lse, float(np.abs(to_f64(lse) - ref_lse).max()))
    torch.cuda.synchronize()
    assert cache.status() == binding.KVF_OK and len(cache) == total
    assert worst <= TOL["bf16"][0] and worst_lse <= 2e-2, (worst, worst_lse)


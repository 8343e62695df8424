"""One launch over many caches (kvf_batch_*): per member the same cache bits as its own
kvf_fold_step, outputs within tolerance of the fp64 oracle."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2605_12471_b200 import binding, workloads
from tests.chain import TOL, to_f64

pytestmark = pytest.mark.gpu

W = workloads.Workload("batch_llama_bf16", 32, 8, 128, "bf16", 256, 1024, 500000.0)


def make_members(n_caches, capacity, max_chunk, seed, spare_pages=3, fill=0x7FC0):
    """n_caches paged caches over one pool, their pages dealt from one shuffled deck."""
    cfg = binding.make_config(W.n_q_heads, W.n_kv_heads, W.head_dim, "bf16", capacity, max_chunk, rope_base=W.rope_base)
    per = (capacity + 127) // 128
    n_pool = n_caches * per + spare_pages
    deck = torch.randperm(n_pool, generator=torch.Generator().manual_seed(seed))[:n_caches * per].to(torch.int32)
    tables = deck.view(n_caches, per).cuda()
    pool = torch.empty(binding.paged_pool_bytes(cfg, n_pool), dtype=torch.uint8, device="cuda")
    pool.view(torch.int16).fill_(fill)                      # NaN wherever no row was ever written
    ws = torch.empty(binding.workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    caches = [binding.PagedCache(cfg, pool, n_pool, tables[i], workspace=ws) for i in range(n_caches)]
    return cfg, pool, tables, caches


def batch_inputs(n_caches, n, seed, step):
    qs, ks, vs = zip(*[workloads.chunk_inputs(W, seed, step, sequence=i, device="cuda", n_tokens=n) for i in range(n_caches)])
    return torch.stack(qs).contiguous(), torch.stack(ks).contiguous(), torch.stack(vs).contiguous()


def test_batch_gives_each_member_its_own_fold_step():
    """Three caches, chunks of mixed length (two row tiles, one tile, decode-shaped, ragged): the pool
    ends up bit-identical to folding each cache by itself, outputs agree with the oracle."""
    chunks = [256, 100, 16, 1, 300, 128, 7]
    total = sum(chunks)
    B = 3
    cfg, pool, tables, caches = make_members(B, total, max(chunks), seed=11)
    _, pool1, _, singles = make_members(B, total, max(chunks), seed=11)
    batch = binding.Batch(caches)
    ocs = [oracle.OracleCache(W.n_q_heads, W.n_kv_heads, W.head_dim, total, rope_base=W.rope_base) for _ in range(B)]
    worst, worst_lse, worst_pair = 0.0, 0.0, 0.0
    for t, n in enumerate(chunks):
        q, k, v = batch_inputs(B, n, 31, t)
        lse = torch.empty((B, n, W.n_q_heads), dtype=torch.float32, device="cuda")
        out = batch.fold_step(q, k, v, lse=lse)
        assert out.shape == q.shape
        rows = sorted({0, n // 2, n - 1})
        for i in range(B):
            alone = singles[i].fold_step(q[i], k[i], v[i])
            worst_pair = max(worst_pair, float((out[i].float() - alone.float()).abs().max()))
            ref, ref_lse, _ = ocs[i].fold_step(to_f64(q[i]), to_f64(k[i]), to_f64(v[i]), rows=rows, want_stats=True)
            worst = max(worst, float(np.abs(to_f64(out[i][rows]) - ref).max()))
            worst_lse = max(worst_lse, float(np.abs(to_f64(lse[i][rows]) - ref_lse).max()))
        assert all(len(c) == sum(chunks[:t + 1]) for c in caches)
    torch.cuda.synchronize()
    assert batch.status_word() == 0
    assert torch.equal(pool, pool1)                          # every page, every row, same bits
    assert worst <= TOL["bf16"][0] and worst_lse <= 2e-2, (worst, worst_lse)
    assert worst_pair <= 2 ** -5                             # two roundings to bf16 of values below 8
    # 3 kernels per step at most, whatever the number of members
    assert batch.launch_count() <= 3 * len(chunks)


def test_batch_of_two_caches_still_cuts_the_key_range():
    """Few members on a long prefix: the plan cuts the (KV head, key tile) line into more ranges than
    KV heads, so every member leaves partial results that the combine kernel merges per member."""
    B, P, n = 2, 8192, 256
    cfg, pool, tables, caches = make_members(B, P + 2 * n, 2048, seed=12)
    batch = binding.Batch(caches)
    ocs = [oracle.OracleCache(W.n_q_heads, W.n_kv_heads, W.head_dim, P + 2 * n, rope_base=W.rope_base) for _ in range(B)]
    for t in range(P // 2048):
        q, k, v = batch_inputs(B, 2048, 41, t)
        batch.fold_step(q, k, v)
        for i in range(B):
            ocs[i].fold_step(to_f64(q[i]), to_f64(k[i]), to_f64(v[i]), rows=[])
    plan = batch.plan(n)
    assert plan[3] == 3 and 4 * W.n_kv_heads * B < plan[2] <= 148      # 4 row pairs per member
    worst = 0.0
    for t in range(2):
        q, k, v = batch_inputs(B, n, 42, t)
        out = batch.fold_step(q, k, v)
        rows = [0, 1, 127, 128, 255]
        for i in range(B):
            ref = ocs[i].fold_step(to_f64(q[i]), to_f64(k[i]), to_f64(v[i]), rows=rows)
            worst = max(worst, float(np.abs(to_f64(out[i][rows]) - ref).max()))
    torch.cuda.synchronize()
    assert batch.status_word() == 0
    assert worst <= TOL["bf16"][0], worst


def test_batch_of_forty_caches_prefill_then_decode_steps():
    """Forty members (5120 CTAs in the prefill launch), then decode-shaped steps of 1 and 8 tokens:
    three sampled members against the oracle, all members' lengths in step."""
    B = 40
    chunks = [1000, 1, 1, 8, 1]
    total = sum(chunks)
    cfg, pool, tables, caches = make_members(B, 1152, 1024, seed=13)
    batch = binding.Batch(caches)
    sample = [0, 17, 39]
    ocs = {i: oracle.OracleCache(W.n_q_heads, W.n_kv_heads, W.head_dim, 1152, rope_base=W.rope_base) for i in sample}
    worst = 0.0
    for t, n in enumerate(chunks):
        q, k, v = batch_inputs(B, n, 51, t)
        out = batch.fold_step(q, k, v)
        rows = sorted({0, n // 3, n - 1})
        for i in sample:
            ref = ocs[i].fold_step(to_f64(q[i]), to_f64(k[i]), to_f64(v[i]), rows=rows)
            worst = max(worst, float(np.abs(to_f64(out[i][rows]) - ref).max()))
    torch.cuda.synchronize()
    assert batch.status_word() == 0 and all(len(c) == total for c in caches)
    assert worst <= TOL["bf16"][0], worst


def test_batch_rejects_members_it_cannot_fold_together():
    cfg, pool, tables, caches = make_members(2, 1024, 256, seed=14)
    flat = binding.Cache(cfg)
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.KvfError) as e:
        binding.Batch([caches[0], flat])
    assert e.value.code == binding.KVF_ERR_UNSUPPORTED                  # a member that is not paged
    with pytest.raises(binding.KvfError) as e:
        binding.Batch([caches[0], caches[0]])
    assert e.value.code == binding.KVF_ERR_INVALID_ARG                  # the same cache twice
    with pytest.raises(binding.KvfError) as e:
        binding.Batch(caches, workspace=ws)
    assert e.value.code == binding.KVF_ERR_CAPACITY                     # workspace too small
    batch = binding.Batch(caches)
    q, k, v = batch_inputs(2, 16, 61, 0)
    caches[1].fold_step(q[1], k[1], v[1])                               # one member runs ahead
    with pytest.raises(binding.KvfError) as e:
        batch.fold_step(q, k, v)
    assert e.value.code == binding.KVF_ERR_INVALID_ARG
    assert len(caches[0]) == 0 and len(caches[1]) == 16                 # nothing was launched
    caches[0].fold_step(q[0], k[0], v[0])
    batch.fold_step(q, k, v)                                            # level again
    torch.cuda.synchronize()
    assert batch.status_word() == 0 and len(caches[0]) == len(caches[1]) == 32


def test_ragged_batch_members_of_different_length():
    """Five sequences of different length taken forward together: a common prompt-sized step each on
    its own first, then decode-shaped and chunk-sized batch steps; every member against its oracle,
    and the pool bit-identical to folding every member by itself."""
    B = 5
    lens0 = [0, 130, 1000, 257, 4000]
    steps = [1, 1, 16, 256, 1, 100]
    cap = max(lens0) + sum(steps) + 128
    cfg, pool, tables, caches = make_members(B, cap, 2048, seed=15)
    _, pool1, _, singles = make_members(B, cap, 2048, seed=15)
    ocs = [oracle.OracleCache(W.n_q_heads, W.n_kv_heads, W.head_dim, cap, rope_base=W.rope_base) for _ in range(B)]
    for i, L in enumerate(lens0):                              # bring the members to different lengths
        t0 = 0
        while t0 < L:
            n = min(2048, L - t0)
            q, k, v = workloads.chunk_inputs(W, 91, t0, sequence=i, device="cuda", n_tokens=n)
            caches[i].fold_step(q, k, v)
            singles[i].fold_step(q, k, v)
            ocs[i].fold_step(to_f64(q), to_f64(k), to_f64(v), rows=[])
            t0 += n
    batch = binding.Batch(caches)
    with pytest.raises(binding.KvfError) as e:
        batch.fold_step(*batch_inputs(B, 1, 92, 0))            # the lock-step call refuses unequal members
    assert e.value.code == binding.KVF_ERR_INVALID_ARG
    worst, worst_lse = 0.0, 0.0
    for t, n in enumerate(steps):
        q, k, v = batch_inputs(B, n, 93, t)
        lse = torch.empty((B, n, W.n_q_heads), dtype=torch.float32, device="cuda")
        out = batch.fold_step(q, k, v, lse=lse, ragged=True)
        rows = sorted({0, n // 2, n - 1})
        for i in range(B):
            singles[i].fold_step(q[i], k[i], v[i])
            ref, ref_lse, _ = ocs[i].fold_step(to_f64(q[i]), to_f64(k[i]), to_f64(v[i]), rows=rows, want_stats=True)
            worst = max(worst, float(np.abs(to_f64(out[i][rows]) - ref).max()))
            worst_lse = max(worst_lse, float(np.abs(to_f64(lse[i][rows]) - ref_lse).max()))
        assert [len(c) for c in caches] == [L + sum(steps[:t + 1]) for L in lens0]
    torch.cuda.synchronize()
    assert batch.status_word() == 0
    assert torch.equal(pool, pool1)
    assert worst <= TOL["bf16"][0] and worst_lse <= 2e-2, (worst, worst_lse)
    # explicit positions: a member may be rotated from another origin than its length
    q, k, v = batch_inputs(B, 1, 94, 0)
    shifted = [len(c) + 7 for c in caches]
    out = batch.fold_step(q, k, v, pos0=shifted, ragged=True)
    for i in (0, 4):
        ref = ocs[i].fold_step(to_f64(q[i]), to_f64(k[i]), to_f64(v[i]), pos0=shifted[i])
        assert float(np.abs(to_f64(out[i]) - ref).max()) <= TOL["bf16"][0]
    caches[0].set_window(4, 64)
    for c in caches[1:]:
        c.set_window(4, 64)
    with pytest.raises(binding.KvfError) as e:
        batch.fold_step(q, k, v, ragged=True)
    assert e.value.code == binding.KVF_ERR_UNSUPPORTED


def test_batch_status_word_written_from_the_host_is_read_back():
    """The batch's own status word, planted by the test (no device-side wait is made to give up)."""
    cfg, pool, tables, caches = make_members(2, 512, 256, seed=17)
    batch = binding.Batch(caches)
    q, k, v = batch_inputs(2, 256, 41, 0)
    batch.fold_step(q, k, v)
    torch.cuda.synchronize()
    assert batch.status_word() == 0
    word = 5 | (22 << 8) | (9 << 16) | (1 << 24)
    batch.workspace[:4].view(torch.int32).fill_(word)
    torch.cuda.synchronize()
    got = batch.status_word()
    assert got == word and (got & 0xFF) == binding.KVF_ERR_TIMEOUT
    assert ((got >> 8) & 0xFF, (got >> 16) & 0xFF, (got >> 24) & 1) == (22, 9, 1)
    assert all(c.status() == binding.KVF_OK for c in caches)        # the members' own words are untouched
    batch.workspace[:4].zero_()
    torch.cuda.synchronize()
    assert batch.status_word() == 0


def test_members_take_steps_of_different_length_and_sit_steps_out():
    """kvf_batch_fold_step_varlen: sequences served together end at different times - one still folds a
    question chunk while others decode single tokens or have finished (n = 0).  Per member the pool ends
    up bit-identical to folding that member by itself, outputs agree with the oracle, blocks of members
    that sit a step out are left alone."""
    B = 4
    total = 1024
    cfg, pool, tables, caches = make_members(B, total, 256, seed=19)
    _, pool1, _, singles = make_members(B, total, 256, seed=19)
    batch = binding.Batch(caches)
    ocs = [oracle.OracleCache(W.n_q_heads, W.n_kv_heads, W.head_dim, total, rope_base=W.rope_base) for _ in range(B)]
    # (max_tokens of the step, tokens of each member)
    steps = [(256, [256, 200, 256, 130]),      # ragged prefill: two row tiles for some, one and a bit for others
             (100, [100, 1, 0, 33]),           # a question chunk, a decoded token, a finished sequence, a short chunk
             (1, [1, 1, 0, 1]),                # decode
             (40, [0, 40, 0, 7]),
             (256, [1, 0, 256, 0]),            # a long chunk beside a single token
             (30, [30, 30, 30, 30])]
    worst, worst_lse, worst_pair = 0.0, 0.0, 0.0
    for t, (mx, ns) in enumerate(steps):
        q, k, v = batch_inputs(B, mx, 43, t)
        out = torch.full(q.shape, 7.0, dtype=torch.bfloat16, device="cuda")
        lse = torch.full((B, mx, W.n_q_heads), 7.0, dtype=torch.float32, device="cuda")
        before = [len(c) for c in caches]
        batch.fold_step_varlen(q, k, v, ns, out=out, lse=lse)
        for i, n in enumerate(ns):
            assert len(caches[i]) == before[i] + n
            # rows past a member's own count (and the whole block of a member that sat out) are untouched
            assert bool((out[i, n:] == 7.0).all()) and bool((lse[i, n:] == 7.0).all())
            if n == 0:
                continue
            alone = singles[i].fold_step(q[i, :n].contiguous(), k[i, :n].contiguous(), v[i, :n].contiguous())
            worst_pair = max(worst_pair, float((out[i, :n].float() - alone.float()).abs().max()))
            rows = sorted({0, n // 2, n - 1})
            ref, ref_lse, _ = ocs[i].fold_step(to_f64(q[i, :n]), to_f64(k[i, :n]), to_f64(v[i, :n]), rows=rows, want_stats=True)
            worst = max(worst, float(np.abs(to_f64(out[i, :n][rows]) - ref).max()))
            worst_lse = max(worst_lse, float(np.abs(to_f64(lse[i, :n][rows]) - ref_lse).max()))
    torch.cuda.synchronize()
    assert batch.status_word() == 0 and all(c.status() == binding.KVF_OK for c in caches)
    assert torch.equal(pool.view(torch.int16), pool1.view(torch.int16))            # every appended row, page for page
    assert worst <= TOL["bf16"][0] and worst_pair <= TOL["bf16"][0] and worst_lse <= 2e-2, (worst, worst_pair, worst_lse)
    # argument checks: a count above the stride, a negative count, a step nobody takes
    lib = binding.load()
    q, k, v = batch_inputs(B, 8, 43, 99)
    out = torch.empty_like(q)

    def call(ns, mx):
        arr = (ctypes.c_int32 * B)(*ns)
        return lib.kvf_batch_fold_step_varlen(batch._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), arr, mx, None,
                                              out.data_ptr(), None, None)
    lens = [len(c) for c in caches]
    assert call([9, 1, 1, 1], 8) == binding.KVF_ERR_INVALID_ARG
    assert call([-1, 1, 1, 1], 8) == binding.KVF_ERR_INVALID_ARG
    assert call([0, 0, 0, 0], 8) == binding.KVF_ERR_INVALID_ARG
    assert call([1, 1, 1, 1], 0) == binding.KVF_ERR_INVALID_ARG
    assert [len(c) for c in caches] == lens

"""Parity of the CUDA fold step (through the C ABI) against the fp64 oracle, small and mid sizes.

Every test here needs a B200; the oracle side runs on the host cores.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2605_12471_b200 import binding, workloads
from tests.chain import TOL, assert_within, run_chain, to_f64

pytestmark = pytest.mark.gpu

SMALL_LLAMA = workloads.Workload("small_llama_bf16", 32, 8, 128, "bf16", 256, 1024, 500000.0)
SMALL_LLAMA_F32 = SMALL_LLAMA.with_(name="small_llama_f32", dtype="f32")


def test_library_is_loaded_from_the_tree():
    lib = binding.load()
    assert lib._name == binding.LIB_PATH


# ------------------------------------------------------------------ config 1
def test_tiny_fold_fp32_matches_oracle_everywhere():
    w = workloads.TINY
    res, cache, oc, _ = run_chain(w, [w.chunk] * w.n_steps, seed=1)
    assert len(cache) == w.tokens == len(oc)
    assert res.count == w.tokens * w.n_q_heads * w.head_dim
    assert_within(res, "f32", "tiny fold")
    assert res.lse_max_abs <= 1e-5


def test_tiny_fold_len_after_t_steps_is_t_times_c():
    w = workloads.TINY
    cache = binding.cache_for(w)
    for t in range(w.n_steps):
        q, k, v = workloads.chunk_inputs(w, 2, t, device="cuda")
        cache.fold_step(q, k, v)
        assert len(cache) == (t + 1) * w.chunk          # host counter, no sync needed
    torch.cuda.synchronize()


@pytest.mark.parametrize("C", [1, 3, 64, 100, 512])
def test_tiny_fold_every_chunking_gives_the_same_outputs(C):
    """fold(C) == fold(C') == one causal pass: the defining invariant, on the GPU."""
    w = workloads.TINY
    q, k, v = workloads.sequence_inputs(w, 3, device="cuda")
    T = w.tokens
    cache = binding.cache_for(w, max_chunk=T)
    ref = cache.fold_step(q, k, v).clone()              # monolithic: one step over everything
    cache.reset()
    outs = []
    for t0 in range(0, T, C):
        outs.append(cache.fold_step(q[t0:t0 + C], k[t0:t0 + C], v[t0:t0 + C]).clone())
    got = torch.cat(outs)
    assert len(cache) == T
    assert (got - ref).abs().max().item() <= 2e-6


# ------------------------------------------------------------ cache contents
def _ulp_diff_bf16(a: torch.Tensor, b: torch.Tensor) -> torch.Tensor:
    ia = a.view(torch.int16).to(torch.int32)
    ib = b.view(torch.int16).to(torch.int32)
    # sign-magnitude -> monotone integers
    ia = torch.where(ia < 0, -(ia & 0x7FFF), ia)
    ib = torch.where(ib < 0, -(ib & 0x7FFF), ib)
    return (ia - ib).abs()


@pytest.mark.parametrize("w,chunks,flags", [
    (workloads.TINY, [64] * 4, 0),
    (workloads.TINY, [33, 1, 94], binding.KVF_ROPE_INTERLEAVED),
    (SMALL_LLAMA, [256, 256, 100, 1], 0),
    (SMALL_LLAMA, [129, 300], binding.KVF_ROPE_INTERLEAVED),
])
def test_appended_cache_bits_match_dtype_faithful_rotation(w, chunks, flags):
    """K rows are the oracle's same-dtype rotation bit for bit; V rows are the inputs verbatim.

    cos/sin come from the device's fp64 routines, which may differ from the host libm by an ulp
    of fp64 and so, after rounding to fp32, in rare table entries: the contract is <= 1 ulp of
    the cache dtype per element with at most 1e-5 of the elements differing at all.
    """
    total = sum(chunks)
    pos_base = 100000                                   # large positions: worst case for the table
    cache = binding.cache_for(w, capacity=total, max_chunk=max(chunks), flags=flags)
    tab = oracle.inv_freq(w.rope_base, w.head_dim)
    ks, vs = [], []
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(w, 5, t, device="cuda", n_tokens=n)
        cache.fold_step(q, k, v, pos0=pos_base + len(cache))
        ks.append(k)
        vs.append(v)
    torch.cuda.synchronize()
    k_all, v_all = torch.cat(ks).cpu(), torch.cat(vs).cpu()
    want = oracle.rope_faithful(k_all.float().numpy(), pos_base, tab,
                                interleaved=bool(flags & binding.KVF_ROPE_INTERLEAVED),
                                to_bf16=(w.dtype == "bf16"))
    want = torch.from_numpy(want).to(k_all.dtype).permute(1, 0, 2).contiguous()     # [Hkv, T, d]
    got_k = cache.k_plane()[:, :total].cpu()
    got_v = cache.v_plane()[:, :total].cpu()
    assert torch.equal(got_v.view(torch.uint8), v_all.permute(1, 0, 2).contiguous().view(torch.uint8))
    if w.dtype == "bf16":
        diff = _ulp_diff_bf16(got_k, want)
    else:
        diff = (got_k.view(torch.int32).to(torch.int64) - want.view(torch.int32).to(torch.int64)).abs()
    assert int(diff.max()) <= 1
    assert float((diff != 0).float().mean()) <= 1e-5
    assert len(cache) == total


def test_prefix_rows_are_untouched_by_later_steps():
    w = SMALL_LLAMA
    cache = binding.cache_for(w, capacity=1024 + 128)
    q, k, v = workloads.chunk_inputs(w, 6, 0, device="cuda", n_tokens=200)
    cache.fold_step(q, k, v)
    torch.cuda.synchronize()
    k0 = cache.k_plane()[:, :200].clone()
    v0 = cache.v_plane()[:, :200].clone()
    for t in range(1, 4):
        q, k, v = workloads.chunk_inputs(w, 6, t, device="cuda")
        cache.fold_step(q, k, v)
    torch.cuda.synchronize()
    assert torch.equal(cache.k_plane()[:, :200], k0)
    assert torch.equal(cache.v_plane()[:, :200], v0)


# -------------------------------------------------------- mid-size parity, both paths
@pytest.mark.parametrize("flags", [0, binding.KVF_FORCE_SIMT])
def test_small_llama_bf16_matches_oracle(flags):
    w = SMALL_LLAMA
    res, cache, _, _ = run_chain(w, [256] * 4, seed=7, flags=flags)
    assert_within(res, "bf16", f"small llama bf16 flags={flags}")
    assert res.lse_max_abs <= 2e-2


@pytest.mark.parametrize("flags", [0, binding.KVF_FORCE_SIMT], ids=["tensor_cores_fp16_halves", "cuda_cores"])
def test_small_llama_f32_matches_oracle(flags):
    """fp32 caches, head_dim 128: the tensor-core kernel on fp16 halves of the operands (three MMAs per
    product, output summed in fp32 registers) and the CUDA-core kernel both meet 1e-5."""
    res, cache, _, _ = run_chain(SMALL_LLAMA_F32, [256] * 3, seed=8, flags=flags)
    assert cache.plan(256, 512)[0] == (0 if flags else 1)
    assert_within(res, "f32", f"small llama f32 flags={flags}")
    assert res.lse_max_abs <= 1e-5


def test_f32_tensor_core_path_on_a_deeper_ragged_chain_with_small_and_large_inputs():
    """Chunks that leave ragged tails in the 64-key steps and the 128-row blocks, a prefix deep enough
    for split key ranges, and inputs scaled down (1/sqrt(128), as the 16K configuration) and up (x 2):
    the split into fp16 halves keeps an absolute 2^-25 on small elements and 22 bits on large ones.
    (Inputs twice as large make logits four times and values twice as large: the absolute bound is
    scaled by that factor of eight.)"""
    for scale, seed in ((1.0, 41), (128 ** -0.5, 42), (2.0, 43)):
        w = SMALL_LLAMA_F32.with_(name=f"f32_ragged_{scale:.3f}", tokens=8192, input_scale=scale)
        chunks = [2048, 1000, 333, 256, 65, 64, 63, 1, 129, 2048, 31, 700]
        check = [1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11]
        res, cache, _, _ = run_chain(w, chunks, seed=seed, check_steps=check, rows_per_step=6)
        assert cache.plan(256, 4096)[0] == 1
        tol = TOL["f32"][0] * max(1.0, scale ** 3)
        assert res.count > 0 and res.max_abs <= tol, (scale, res.max_abs, res.per_step)
        assert res.lse_max_abs <= 1e-5 * max(1.0, scale * scale)


def test_f32_tensor_core_path_flags_magnitudes_beyond_fp16_range():
    """A key element of 1e5 cannot be split into fp16 halves: the step still runs to its end and the
    status word says KVF_ERR_RANGE; the CUDA-core kernel takes the same inputs without complaint."""
    w = SMALL_LLAMA_F32.with_(name="f32_range")
    q, k, v = workloads.chunk_inputs(w, 44, 0, device="cuda")
    k[3, 2, 17] = 1.0e5
    cache = binding.cache_for(w)
    cache.fold_step(q, k, v)
    torch.cuda.synchronize()
    assert cache.status() == binding.KVF_ERR_RANGE and (cache.status_word() & 0xFF) == 7
    assert binding.load().kvf_status_str(cache.status()).decode() == "KVF_ERR_RANGE"
    simt = binding.cache_for(w, flags=binding.KVF_FORCE_SIMT)
    out = simt.fold_step(q, k, v)
    torch.cuda.synchronize()
    assert simt.status() == binding.KVF_OK and torch.isfinite(out).all()
    # (a logit of order 1e5 carries an fp32 rounding error of order 1e-2, so the rows that see that key are
    # only as close to the oracle as fp32 allows)
    oc = oracle.OracleCache(w.n_q_heads, w.n_kv_heads, w.head_dim, w.chunk, rope_base=w.rope_base)
    ref = oc.fold_step(to_f64(q), to_f64(k), to_f64(v))
    assert np.abs(to_f64(out[:3]) - ref[:3]).max() <= TOL["f32"][0]      # rows before the large key
    assert np.abs(to_f64(out) - ref).max() <= 1e-2


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_ragged_chunk_lengths_including_single_tokens(dtype):
    w = SMALL_LLAMA.with_(name=f"ragged_{dtype}", dtype=dtype)
    chunks = [1, 1, 31, 32, 33, 127, 129, 255, 1, 64, 7]
    res, cache, _, _ = run_chain(w, chunks, seed=9)
    assert len(cache) == sum(chunks)
    assert_within(res, dtype, "ragged")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_out_f32_flag_and_interleaved_rotation(dtype):
    w = SMALL_LLAMA.with_(name=f"flags_{dtype}", dtype=dtype)
    flags = binding.KVF_OUT_F32 | binding.KVF_ROPE_INTERLEAVED
    res, cache, _, outs = run_chain(w, [200, 56, 256], seed=10, flags=flags, keep_outputs=True)
    assert outs[0].dtype == torch.float32
    assert_within(res, dtype, "out_f32+interleaved")


@pytest.mark.parametrize("dtype,flags", [("bf16", 0), ("bf16", binding.KVF_FORCE_SIMT), ("f32", 0),
                                         ("f32", binding.KVF_FORCE_SIMT)])
def test_split_counts_agree_with_each_other_and_with_the_oracle(dtype, flags):
    w = SMALL_LLAMA.with_(name=f"split_{dtype}", dtype=dtype, tokens=4096)
    chunks = [2048, 256, 100, 1, 64]
    ref = None
    for splits in (1, 2, 5, 0):
        res, cache, _, outs = run_chain(w, chunks, seed=11, flags=flags, splits=splits,
                                        check_steps=[1, 2, 3, 4], rows_per_step=4, keep_outputs=True)
        assert_within(res, dtype, f"splits={splits}")
        last = torch.cat([o.float().flatten() for o in outs[1:]])
        if ref is None:
            ref = last
        else:
            assert (last - ref).abs().max().item() <= TOL[dtype][0]
        if splits in (2, 5):
            assert cache.plan(64)[1] == splits


def test_results_are_bitwise_reproducible():
    w = SMALL_LLAMA.with_(name="determinism", tokens=2048)
    a = run_chain(w, [512, 256, 256, 3], seed=12, check_steps=[], keep_outputs=True)[3]
    b = run_chain(w, [512, 256, 256, 3], seed=12, check_steps=[], keep_outputs=True)[3]
    for x, y in zip(a, b):
        assert torch.equal(x.view(torch.int16), y.view(torch.int16))


def test_non_continued_positions_are_honoured():
    """pos0 is used for the rotation only; the oracle gets the same positions."""
    w = SMALL_LLAMA.with_(name="positions")
    res, _, _, _ = run_chain(w, [128, 128, 64], seed=13, positions=[1000, 50000, 7])
    assert_within(res, "bf16", "free positions")


def test_uninitialised_storage_with_nan_bits_does_not_leak():
    """Rows past the end of the cache are not content: non-finite garbage there must not matter."""
    w = SMALL_LLAMA.with_(name="nan_storage")
    cache = binding.cache_for(w, capacity=1000, max_chunk=300)
    cache.storage.view(torch.int16).fill_(0x7FC0)   # bf16 NaN
    oc = oracle.OracleCache(w.n_q_heads, w.n_kv_heads, w.head_dim, 1000, rope_base=w.rope_base)
    for t, n in enumerate([70, 300, 1]):
        q, k, v = workloads.chunk_inputs(w, 14, t, device="cuda", n_tokens=n)
        out = cache.fold_step(q, k, v)
        ref = oc.fold_step(to_f64(q), to_f64(k), to_f64(v))
        assert torch.isfinite(out).all()
        assert np.abs(to_f64(out) - ref).max() <= TOL["bf16"][0]


def test_planted_key_survives_the_chain():
    """Kernel-level needle: a key planted in chunk 0 is recovered by a query 31 chunks later."""
    w = SMALL_LLAMA.with_(name="needle", tokens=8192)
    H, Hkv, d, C = w.n_q_heads, w.n_kv_heads, w.head_dim, 256
    cache = binding.cache_for(w, capacity=8192, max_chunk=C)
    needle_v = None
    tab = torch.from_numpy(oracle.inv_freq(w.rope_base, d))

    def unrotate(vec, pos):
        ang = pos * tab
        lo, hi = vec[:d // 2].double(), vec[d // 2:].double()
        return torch.cat([lo * torch.cos(ang) + hi * torch.sin(ang), hi * torch.cos(ang) - lo * torch.sin(ang)])

    direction = torch.zeros(d)
    direction[:4] = 0.5                                   # |direction| = 1
    for t in range(32):
        q, k, v = workloads.chunk_inputs(w, 15, t, device="cuda")
        q, k = q * 0.05, k * 0.05
        if t == 0:
            k[5] = unrotate(direction * 40.0, 5).to(k.dtype).to("cuda")
            needle_v = v[5].clone()
        if t == 31:
            q[200] = unrotate(direction * 40.0, 31 * C + 200).to(q.dtype).to("cuda")
        out = cache.fold_step(q.contiguous(), k.contiguous(), v)
    for h in range(H):
        assert (out[200, h].float() - needle_v[h // 4].float()).abs().max().item() <= 2e-2


# ------------------------------------------------------------------ host-side errors
def test_errors_are_return_codes_and_change_nothing():
    w = SMALL_LLAMA
    cfg = binding.make_config(32, 8, 128, "bf16", 512, 256, rope_base=5e5, flags=binding.KVF_STRICT_POS)
    cache = binding.Cache(cfg)
    q, k, v = workloads.chunk_inputs(w, 16, 0, device="cuda")
    lib = binding.load()
    out = torch.empty_like(q)
    h = cache._h

    def call(qp, kp, vp, n, pos0, op):
        return lib.kvf_fold_step(h, qp, kp, vp, n, pos0, op, None, None)

    launches = cache.launch_count()
    assert call(None, k.data_ptr(), v.data_ptr(), 256, 0, out.data_ptr()) == binding.KVF_ERR_INVALID_ARG
    assert call(q.data_ptr() + 2, k.data_ptr(), v.data_ptr(), 256, 0, out.data_ptr()) == binding.KVF_ERR_INVALID_ARG
    assert call(q.data_ptr(), k.data_ptr(), v.data_ptr(), 0, 0, out.data_ptr()) == binding.KVF_ERR_INVALID_ARG
    assert call(q.data_ptr(), k.data_ptr(), v.data_ptr(), 257, 0, out.data_ptr()) == binding.KVF_ERR_INVALID_ARG
    assert call(q.data_ptr(), k.data_ptr(), v.data_ptr(), 256, 5, out.data_ptr()) == binding.KVF_ERR_POS
    assert len(cache) == 0 and cache.launch_count() == launches
    cache.fold_step(q, k, v)
    cache.fold_step(q, k, v)
    assert len(cache) == 512
    assert call(q.data_ptr(), k.data_ptr(), v.data_ptr(), 1, 512, out.data_ptr()) == binding.KVF_ERR_CAPACITY
    assert len(cache) == 512
    with pytest.raises(binding.KvfError):
        cache.fold_step(q, k, v)
    cache.reset()
    assert len(cache) == 0
    assert lib.kvf_cache_len(None) == -1
    torch.cuda.synchronize()
    assert cache.status() == binding.KVF_OK


def test_status_word_written_from_the_host_is_reported_as_a_timed_out_wait():
    """The path a bounded device-side wait takes when it gives up, without making any wait give up:
    the test itself writes the word such a wait would leave (low byte 5 = timeout, then barrier 22,
    warp 9, parity 1) into the cache's workspace and reads it back through the two entry points."""
    lib = binding.load()
    cache = binding.cache_for(SMALL_LLAMA)
    q, k, v = workloads.chunk_inputs(SMALL_LLAMA, 40, 0, device="cuda")
    cache.fold_step(q, k, v)
    torch.cuda.synchronize()
    assert cache.status() == binding.KVF_OK and cache.status_word() == 0
    word = 5 | (22 << 8) | (9 << 16) | (1 << 24)
    cache.workspace[:4].view(torch.int32).fill_(word)
    torch.cuda.synchronize()
    assert cache.status() == binding.KVF_ERR_TIMEOUT
    assert lib.kvf_status_str(cache.status()).decode() == "KVF_ERR_TIMEOUT"
    got = cache.status_word()
    assert got == word
    assert (got & 0xFF, (got >> 8) & 0xFF, (got >> 16) & 0xFF, (got >> 24) & 1) == (5, 22, 9, 1)
    # the word is sticky until the owner of the workspace clears it; steps still run
    cache.fold_step(q, k, v)
    torch.cuda.synchronize()
    assert cache.status() == binding.KVF_ERR_TIMEOUT and len(cache) == 2 * SMALL_LLAMA.chunk
    cache.workspace[:4].zero_()
    torch.cuda.synchronize()
    assert cache.status() == binding.KVF_OK and cache.status_word() == 0


def test_create_rejects_short_or_misaligned_buffers():
    lib = binding.load()
    cfg = binding.make_config(32, 8, 128, "bf16", 512, 256, rope_base=5e5)
    sb, wb = binding.cache_storage_bytes(cfg), binding.workspace_bytes(cfg)
    st = torch.empty(sb + 512, dtype=torch.uint8, device="cuda")
    ws = torch.empty(wb + 512, dtype=torch.uint8, device="cuda")
    h = ctypes.c_void_p()
    assert lib.kvf_cache_create(ctypes.byref(cfg), st.data_ptr(), sb - 1, ws.data_ptr(), wb, ctypes.byref(h)) == binding.KVF_ERR_CAPACITY
    assert lib.kvf_cache_create(ctypes.byref(cfg), st.data_ptr(), sb, ws.data_ptr(), wb - 1, ctypes.byref(h)) == binding.KVF_ERR_CAPACITY
    assert lib.kvf_cache_create(ctypes.byref(cfg), st.data_ptr() + 16, sb, ws.data_ptr(), wb, ctypes.byref(h)) == binding.KVF_ERR_INVALID_ARG
    assert lib.kvf_cache_create(ctypes.byref(cfg), st.data_ptr(), sb, ws.data_ptr(), wb, ctypes.byref(h)) == binding.KVF_OK
    lib.kvf_cache_destroy(h)


@pytest.mark.parametrize("flags", [0, binding.KVF_HOST_UPLOAD_AHEAD], ids=["one_stream", "upload_ahead"])
def test_host_buffer_entry_point_matches_device_entry_point(flags):
    w = SMALL_LLAMA
    a = binding.cache_for(w)
    b = binding.cache_for(w, flags=flags)
    for t in range(3):
        q, k, v = workloads.chunk_inputs(w, 17, t, device="cuda")
        want = a.fold_step(q, k, v)
        qh, kh, vh = (x.cpu().pin_memory() for x in (q, k, v))
        oh = torch.empty(want.shape, dtype=want.dtype).pin_memory()
        lh = torch.empty((w.chunk, w.n_q_heads), dtype=torch.float32).pin_memory()
        b.fold_step_host(qh, kh, vh, oh, lse=lh)
        torch.cuda.synchronize()
        assert torch.equal(oh.view(torch.int16), want.cpu().view(torch.int16))
        assert torch.isfinite(lh).all()
    assert len(a) == len(b) == 3 * w.chunk


def test_profile_counters_and_launch_count():
    w = SMALL_LLAMA
    cache = binding.cache_for(w)
    cache.profile(True)
    for t in range(4):
        q, k, v = workloads.chunk_inputs(w, 18, t, device="cuda")
        cache.fold_step(q, k, v)
    ms, cnt = cache.profile_read()
    assert cnt[0] == 4 and cnt[1] == 4
    assert cache.launch_count() == sum(cnt)
    assert all(m >= 0 for m in ms) and ms[1] > 0


def test_attention_kernels_report_the_clock_they_ran_at():
    """kvf_cache_sm_clock: the first CTA of every tensor-core attention launch adds its SM cycles and its
    nanoseconds to two sums; their ratio is a clock between idle and the part's maximum."""
    for w in (SMALL_LLAMA.with_(name="clock_bf16", tokens=4096), SMALL_LLAMA_F32.with_(name="clock_f32", tokens=4096)):
        cache = binding.cache_for(w)
        assert cache.sm_clock() == (0, 0)
        q, k, v = workloads.chunk_inputs(w, 45, 0, device="cuda")
        for t in range(8):
            cache.fold_step(q, k, v)
        cycles, ns = cache.sm_clock()                      # a blocking copy: the steps are done when it returns
        assert cycles > 0 and ns > 0
        mhz = 1e3 * cycles / ns
        assert 300.0 < mhz < 2200.0, mhz                  # (a B200's SM clock tops out at 1965 MHz)
    tiny = binding.cache_for(workloads.TINY)              # CUDA-core kernel: it does not count
    q, k, v = workloads.chunk_inputs(workloads.TINY, 46, 0, device="cuda")
    tiny.fold_step(q, k, v)
    assert tiny.sm_clock() == (0, 0)


# ------------------------------------------------------------------ short chunks at depth
@pytest.mark.parametrize("splits", [0, 1], ids=["merged_ranges", "one_range_per_head"])
def test_decode_shaped_steps_with_fp32_output(splits):
    """One to four tokens per step take the decode kernel; with one key range per KV head it writes the outputs
    and log-sum-exps itself (no merge), otherwise the merge kernel does: both in fp32 under KVF_OUT_F32."""
    w = SMALL_LLAMA.with_(name="decode_out_f32", tokens=4096)
    chunks = [2048, 300, 1, 1, 2, 3, 4, 1]
    res, cache, _, outs = run_chain(w, chunks, seed=23, flags=binding.KVF_OUT_F32, splits=splits,
                                    check_steps=list(range(2, len(chunks))), keep_outputs=True)
    assert outs[-1].dtype == torch.float32
    if splits:
        assert cache.plan(1)[1] == 1
    assert_within(res, "bf16", "decode, fp32 output")
    assert res.lse_max_abs <= 2e-2, res.lse_max_abs


def test_short_chunks_deep_in_a_chain_match_the_oracle():
    """Decode- and question-shaped steps (1 .. 32 tokens: at most one 128-row tile) after a long
    prefix: the kernel deals their key tiles to two streams and always merges partial results."""
    w = SMALL_LLAMA.with_(name="short_chunks_at_depth", tokens=16384)
    chunks = [2048] * 5 + [32] * 6 + [1] * 5 + [16, 31, 32, 7, 2, 32, 33, 64, 5]
    check = list(range(5, len(chunks)))
    res, cache, _, _ = run_chain(w, chunks, seed=19, check_steps=check, rows_per_step=3)
    assert len(cache) == sum(chunks)
    assert cache.plan(32, 10000)[3] == 3 and cache.plan(33, 10000)[1] >= 1
    assert_within(res, "bf16", "short chunks at depth")
    assert res.rel_rms <= 2e-2, res.rel_rms


def test_short_chunk_chains_repeat_bitwise_without_host_synchronisation():
    """The same chain of 32-token steps enqueued three times back to back (reset in between, no
    synchronisation inside a chain) gives the same bits every time."""
    w = SMALL_LLAMA.with_(name="short_chunks_async", tokens=12288 + 32 * 48)
    cache = binding.cache_for(w, max_chunk=2048)
    fq, fk, fv = workloads.chunk_inputs(w.with_(chunk=2048), 20, 0, device="cuda")
    q, k, v = workloads.sequence_inputs(w.with_(tokens=32 * 48, chunk=32), 21, device="cuda")
    outs = []
    for rep in range(3):
        cache.reset()
        for _ in range(6):
            cache.fold_step(fq, fk, fv)
        out = torch.empty_like(q)
        for t in range(48):
            cache.fold_step(q[32 * t:32 * t + 32], k[32 * t:32 * t + 32], v[32 * t:32 * t + 32], out=out[32 * t:32 * t + 32])
        outs.append(out)
    torch.cuda.synchronize()
    assert cache.status() == binding.KVF_OK
    assert torch.isfinite(outs[0].float()).all()
    for o in outs[1:]:
        assert torch.equal(o.view(torch.int16), outs[0].view(torch.int16))


# ------------------------------------------------------------------ paged cache
def test_paged_cache_matches_the_contiguous_cache_and_the_oracle():
    """Rows in 128-token pages scattered over a shared pool: same bits as the contiguous cache
    (the arithmetic does not depend on where a row lives) and within tolerance of the oracle."""
    w = SMALL_LLAMA.with_(name="paged", tokens=4096)
    chunks = [256, 256, 100, 1, 411, 32, 7, 1024, 33, 128, 5]
    total = sum(chunks)
    cfg = binding.make_config(w.n_q_heads, w.n_kv_heads, w.head_dim, "bf16", total, max(chunks), rope_base=w.rope_base)
    n_table = (total + 127) // 128
    n_pool = 2 * n_table + 3
    gen = torch.Generator().manual_seed(5)
    perm = torch.randperm(n_pool, generator=gen)[:n_table].to(torch.int32)        # scattered, not in order
    table = perm.cuda()
    pool = torch.empty(binding.paged_pool_bytes(cfg, n_pool), dtype=torch.uint8, device="cuda")
    pool.view(torch.int16).fill_(0x7FC0)                                          # NaN everywhere a row was never written
    paged = binding.PagedCache(cfg, pool, n_pool, table)
    flat = binding.Cache(cfg)
    oc = oracle.OracleCache(w.n_q_heads, w.n_kv_heads, w.head_dim, total, rope_base=w.rope_base)
    worst = 0.0
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(w, 23, t, device="cuda", n_tokens=n)
        got = paged.fold_step(q, k, v)
        want = flat.fold_step(q, k, v)
        assert torch.equal(got.view(torch.int16), want.view(torch.int16)), f"step {t}"
        ref = oc.fold_step(to_f64(q), to_f64(k), to_f64(v), rows=[0, n - 1])
        worst = max(worst, float(np.abs(to_f64(got[[0, n - 1]]) - ref).max()))
    torch.cuda.synchronize()
    assert len(paged) == total and paged.status() == binding.KVF_OK
    assert worst <= TOL["bf16"][0]
    # the rows are where the table says
    kp, vp = paged.page_rows(0), paged.page_rows(1)
    fk, fv = flat.k_plane(), flat.v_plane()
    for i in (0, 3, n_table - 1):
        rows = min(128, total - 128 * i)
        assert torch.equal(kp[int(perm[i]), :, :rows], fk[:, 128 * i:128 * i + rows])
        assert torch.equal(vp[int(perm[i]), :, :rows], fv[:, 128 * i:128 * i + rows])


def test_paged_cache_rejects_what_it_does_not_cover():
    lib = binding.load()
    cfg32 = binding.make_config(32, 8, 128, "f32", 1024, 256, rope_base=5e5)
    buf = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    table = torch.zeros(8, dtype=torch.int32, device="cuda")
    h = ctypes.c_void_p()
    rc = lib.kvf_paged_cache_create(ctypes.byref(cfg32), buf.data_ptr(), buf.numel(), 1, table.data_ptr(), buf.data_ptr(),
                                    buf.numel(), ctypes.byref(h))
    assert rc == binding.KVF_ERR_UNSUPPORTED
    cfg = binding.make_config(32, 8, 128, "bf16", 1024, 256, rope_base=5e5)
    rc = lib.kvf_paged_cache_create(ctypes.byref(cfg), buf.data_ptr(), buf.numel(), 8, table.data_ptr(), buf.data_ptr(),
                                    buf.numel(), ctypes.byref(h))
    assert rc == binding.KVF_ERR_CAPACITY                     # 8 pages need 4 MiB


def test_host_steps_with_upload_ahead_enqueued_back_to_back():
    """Eight host steps enqueued without any synchronisation in between (each upload overlaps the
    step before it, the staging sets alternate): same bits as the device entry point."""
    w = SMALL_LLAMA.with_(name="upload_ahead", tokens=2048)
    dev = binding.cache_for(w)
    host = binding.cache_for(w, flags=binding.KVF_HOST_UPLOAD_AHEAD)
    want, got, keep = [], [], []
    for t in range(8):
        q, k, v = workloads.chunk_inputs(w, 19, t, device="cuda")
        want.append(dev.fold_step(q, k, v))
        qh, kh, vh = (x.cpu().pin_memory() for x in (q, k, v))
        oh = torch.empty(q.shape, dtype=q.dtype).pin_memory()
        keep.append((qh, kh, vh))
        got.append(oh)
    torch.cuda.synchronize()
    for t in range(8):
        host.fold_step_host(*keep[t], got[t])
    torch.cuda.synchronize()
    assert host.status() == binding.KVF_OK and len(host) == 2048
    for t in range(8):
        assert torch.equal(got[t].view(torch.int16), want[t].cpu().view(torch.int16)), t


@pytest.mark.parametrize("flags", [binding.KVF_HOST_DOWNLOAD_BEHIND,
                                   binding.KVF_HOST_DOWNLOAD_BEHIND | binding.KVF_HOST_UPLOAD_AHEAD],
                         ids=["download_behind", "upload_ahead_and_download_behind"])
def test_host_steps_with_results_copied_behind_the_next_step(flags):
    """Eight host steps enqueued back to back with the result copies on the library's own stream (two
    result staging sets, the copy of step t behind step t+1): the same bits as the device entry point,
    and the relaxed contract - step t's results are there once the stream has passed call t+1, the last
    step's after a flush."""
    w = SMALL_LLAMA.with_(name="download_behind", tokens=2048)
    dev = binding.cache_for(w)
    host = binding.cache_for(w, flags=flags)
    want, got, lses, keep = [], [], [], []
    for t in range(8):
        q, k, v = workloads.chunk_inputs(w, 19, t, device="cuda")
        want.append(dev.fold_step(q, k, v))
        keep.append(tuple(x.cpu().pin_memory() for x in (q, k, v)))
        got.append(torch.zeros(q.shape, dtype=q.dtype).pin_memory())
        lses.append(torch.zeros((w.chunk, w.n_q_heads), dtype=torch.float32).pin_memory())
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()
    for t in range(7):
        host.fold_step_host(*keep[t], got[t], lse=lses[t])
    stream.synchronize()                     # the stream has passed the end of call 6: steps 0 .. 5 are there
    for t in range(6):
        assert torch.equal(got[t].view(torch.int16), want[t].cpu().view(torch.int16)), t
    host.fold_step_host(*keep[7], got[7], lse=lses[7])
    host.host_flush()
    stream.synchronize()
    assert host.status() == binding.KVF_OK and len(host) == 2048
    for t in range(8):
        assert torch.equal(got[t].view(torch.int16), want[t].cpu().view(torch.int16)), t
        assert torch.isfinite(lses[t]).all() and float(lses[t].abs().max()) > 0
    # a flush with nothing outstanding, and on a cache without the flag, is harmless
    host.host_flush()
    dev.host_flush()
    torch.cuda.synchronize()


def _merge_behind_chain(flags, chunks, seed=23):
    """The same chain on a plain cache and on one with KVF_COMBINE_BEHIND (+ flags); steps enqueued back to back."""
    total = sum(chunks)
    w = SMALL_LLAMA.with_(name="merge_behind", tokens=total)
    plain = binding.cache_for(w, capacity=total, max_chunk=max(chunks), flags=flags)
    behind = binding.cache_for(w, capacity=total, max_chunk=max(chunks), flags=flags | binding.KVF_COMBINE_BEHIND)
    ins = [workloads.chunk_inputs(w, seed, t, device="cuda", n_tokens=n) for t, n in enumerate(chunks)]
    want, want_lse = [], []
    for q, k, v in ins:
        lse = torch.empty((q.shape[0], w.n_q_heads), dtype=torch.float32, device="cuda")
        want.append(plain.fold_step(q, k, v, lse=lse))
        want_lse.append(lse)
    torch.cuda.synchronize()
    return w, behind, ins, want, want_lse


@pytest.mark.parametrize("flags", [0, binding.KVF_CACHE_INT8], ids=["bf16", "int8"])
def test_merge_behind_the_attention_kernel_gives_the_same_bits(flags):
    """KVF_COMBINE_BEHIND: the merge of step t runs on the library's stream beside the rotate + append kernel
    of step t+1.  Same bits as without the flag; step t's results are there once the stream has passed call
    t+1, the last step's after a flush.  Chunks of 256 and of one token, at prefixes where the plan has a
    merge kernel and where it has none."""
    chunks = [256] * 6 + [1, 1, 3, 256, 1, 1]
    w, cache, ins, want, want_lse = _merge_behind_chain(flags, chunks)
    kernels = [cache.plan(n, sum(chunks[:t]))[3] for t, n in enumerate(chunks)]
    assert 3 in kernels
    got = [torch.zeros_like(x) for x in want]
    got_lse = [torch.zeros_like(x) for x in want_lse]
    stream = torch.cuda.current_stream()
    last = len(chunks) - 1
    for t in range(last):
        cache.fold_step(*ins[t], out=got[t], lse=got_lse[t])
    stream.synchronize()                     # the stream has passed the end of call last - 1
    for t in range(last - 1):
        assert torch.equal(got[t].view(torch.int16), want[t].view(torch.int16)), t
    cache.fold_step(*ins[last], out=got[last], lse=got_lse[last])
    cache.flush()
    stream.synchronize()
    assert cache.status() == binding.KVF_OK and len(cache) == sum(chunks)
    for t in range(len(chunks)):
        assert torch.equal(got[t].view(torch.int16), want[t].view(torch.int16)), t
        assert torch.equal(got_lse[t], want_lse[t]), t
    cache.flush()                            # nothing outstanding: harmless
    torch.cuda.synchronize()


def test_merge_behind_inside_a_stream_capture():
    """A chain with KVF_COMBINE_BEHIND captured into a CUDA graph (the library's stream joins the capture
    through its events and is joined again by the flush) and replayed: the same bits.  A step that meets a
    merge left open outside its capture is refused and enqueues nothing."""
    chunks = [256] * 8
    w, cache, ins, want, _ = _merge_behind_chain(0, chunks)
    got = [torch.zeros_like(x) for x in want]
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for t in range(len(chunks)):
            cache.fold_step(*ins[t], out=got[t])
        cache.flush()
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    for t in range(len(chunks)):
        assert torch.equal(got[t].view(torch.int16), want[t].view(torch.int16)), t
    # an open merge from before the capture
    cache.reset()
    first = next(t for t in range(len(chunks)) if cache.plan(256, 256 * t)[3] == 3)     # the first step with a merge kernel
    assert first < len(chunks) - 1
    for t in range(first + 1):
        cache.fold_step(*ins[t], out=got[t])
    launches = cache.launch_count()
    refused = torch.cuda.CUDAGraph()
    with torch.cuda.graph(refused):
        with pytest.raises(binding.KvfError) as err:
            cache.fold_step(*ins[first + 1], out=got[first + 1])
        with pytest.raises(binding.KvfError):
            cache.flush()
    assert err.value.code == binding.KVF_ERR_INVALID_ARG
    assert len(cache) == 256 * (first + 1) and cache.launch_count() == launches
    cache.flush()
    torch.cuda.synchronize()
    assert torch.equal(got[first].view(torch.int16), want[first].view(torch.int16))
    assert cache.status() == binding.KVF_OK


def test_merge_behind_with_host_steps_and_results_copied_behind():
    """KVF_COMBINE_BEHIND together with the two host-step flags: the result copy of a step waits for its merge."""
    flags = binding.KVF_HOST_DOWNLOAD_BEHIND | binding.KVF_HOST_UPLOAD_AHEAD
    chunks = [256] * 8
    w, cache, ins, want, want_lse = _merge_behind_chain(flags, chunks)
    keep = [tuple(x.cpu().pin_memory() for x in qkv) for qkv in ins]
    got = [torch.zeros(x.shape, dtype=x.dtype).pin_memory() for x in want]
    lses = [torch.zeros(x.shape, dtype=torch.float32).pin_memory() for x in want_lse]
    torch.cuda.synchronize()
    for t in range(len(chunks)):
        cache.fold_step_host(*keep[t], got[t], lse=lses[t])
    cache.flush()
    torch.cuda.current_stream().synchronize()
    assert cache.status() == binding.KVF_OK
    for t in range(len(chunks)):
        assert torch.equal(got[t].view(torch.int16), want[t].cpu().view(torch.int16)), t
        assert torch.equal(lses[t], want_lse[t].cpu()), t


def test_plan_fills_the_last_wave_when_whole_kv_heads_would_leave_it_half_empty():
    """148 SMs: 32 row pairs x 8 KV heads = 256 CTAs is 1.73 waves, 32 x 9 groups = 288 is 1.95; 128 row
    pairs x 8 = 1024 CTAs (6.9 waves) stays with whole KV heads and needs no combine kernel."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    cache = binding.cache_for(SMALL_LLAMA.with_(name="plan_probe", tokens=65536, chunk=8192), capacity=65536, max_chunk=8192)
    tc, parts, ctas, kernels = cache.plan(2048, 61440)
    if sms == 148:
        assert (tc, ctas, kernels) == (1, 288, 3) and parts == 2
    tc, parts, ctas, kernels = cache.plan(8192, 57344)
    assert (tc, parts, ctas, kernels) == (1, 1, 128 * 8, 2)
    tc, parts, ctas, kernels = cache.plan(256, 130816 - 65536)      # the benchmark's chunk: one CTA per SM
    assert tc == 1 and ctas == (sms // 4) * 4 and kernels == 3
    # a short line: 32 groups (4 per KV head, every CTA inside one KV head) instead of 37 that straddle heads
    tc, parts, ctas, kernels = cache.plan(256, 2048)
    if sms == 148:
        assert (tc, parts, ctas, kernels) == (1, 4, 128, 3)

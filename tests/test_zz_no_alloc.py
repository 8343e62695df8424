"""kvf_fold_step_static: the step whose scratch is a fixed array inside the library.

Some callers may not allocate device memory at all (a server whose memory is already all in its
own pool, a loop that has to stay out of the allocator).  For them the library carries its own
scratch; this file checks that entry point against the ordinary one, call after call, on planes
the test owns.  It is collected last so that a run stopping at the first failure has already
run everything else.
"""
import ctypes

import pytest
import torch

from paper_2605_12471_b200 import binding, workloads
from tests.chain import TOL

pytestmark = pytest.mark.gpu


def _same_chain(w, chunks, seed, flags=0):
    """Fold `chunks` through kvf_fold_step (handle + workspace) and through kvf_fold_step_static
    (raw planes + built-in scratch); compare every step's output, lse and the planes."""
    total = sum(chunks)
    cfg = binding.make_config(w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, total, max(chunks),
                              rope_base=w.rope_base, flags=flags)
    ref = binding.Cache(cfg)
    storage = torch.empty(binding.cache_storage_bytes(cfg), dtype=torch.uint8, device="cuda")
    length = 0
    mx, _ = TOL[w.dtype]
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(w, seed, t, device="cuda", n_tokens=n)
        lse_a = torch.empty((n, w.n_q_heads), dtype=torch.float32, device="cuda")
        lse_b = torch.empty_like(lse_a)
        want = ref.fold_step(q, k, v, lse=lse_a)
        got = torch.empty_like(want)
        binding.fold_step_static(cfg, storage, length, q, k, v, out=got, lse=lse_b)
        length += n
        torch.cuda.synchronize()
        assert torch.isfinite(got.float()).all()
        assert (got.float() - want.float()).abs().max().item() <= mx, f"step {t}"
        assert (lse_a - lse_b).abs().max().item() <= 1e-3, f"step {t} lse"
    assert length == len(ref) == total
    return cfg, ref, storage


def test_static_scratch_step_matches_the_ordinary_step_call_after_call():
    w = workloads.Workload("static_llama", 32, 8, 128, "bf16", 256, 4096, 500000.0)
    # prefix grows past the point where the key range is split; then short and ragged steps
    cfg, ref, storage = _same_chain(w, [512, 512, 512, 512, 256, 256, 64, 64, 1, 100], seed=31)
    plane = storage.numel() // 2
    total = len(ref)
    got_k = storage[:plane].view(torch.bfloat16).view(8, cfg.capacity, 128)[:, :total]
    got_v = storage[plane:].view(torch.bfloat16).view(8, cfg.capacity, 128)[:, :total]
    assert torch.equal(got_k, ref.k_plane()[:, :total])
    assert torch.equal(got_v, ref.v_plane()[:, :total])


def test_static_scratch_step_fp32_and_small_heads():
    w = workloads.TINY
    _same_chain(w, [64, 64, 33, 1, 200], seed=32)


def test_static_scratch_step_fp32_on_the_tensor_cores():
    w = workloads.Workload("static_llama_f32", 32, 8, 128, "f32", 256, 2048, 500000.0)
    _same_chain(w, [256, 256, 256, 256, 100, 1, 64], seed=33)


def test_static_scratch_step_with_groups_of_seven():
    """28 / 4 heads: the fixed scratch holds the partial rows in the padded-group layout as well."""
    w = workloads.Workload("static_qwen", 28, 4, 128, "bf16", 256, 4096, 500000.0)
    _same_chain(w, [512, 512, 256, 256, 19, 2, 1, 100], seed=34)


def test_static_scratch_rejects_sizes_beyond_its_fixed_maximum():
    lib = binding.load()
    cfg = binding.make_config(32, 8, 128, "bf16", 4096, 1024, rope_base=5e5)      # 1024 x 32 x 128 x 2 B = 8 MiB > 4 MiB
    storage = torch.empty(binding.cache_storage_bytes(cfg), dtype=torch.uint8, device="cuda")
    q = torch.zeros((1024, 32, 128), dtype=torch.bfloat16, device="cuda")
    k = torch.zeros((1024, 8, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(q)
    rc = lib.kvf_fold_step_static(ctypes.byref(cfg), storage.data_ptr(), storage.numel(), 0, q.data_ptr(),
                                  k.data_ptr(), k.data_ptr(), 1024, 0, out.data_ptr(), None, None)
    assert rc == binding.KVF_ERR_CAPACITY
    assert b"static scratch" in lib.kvf_last_cuda_error()
    ok = binding.make_config(32, 8, 128, "bf16", 4096, 512, rope_base=5e5)
    rc = lib.kvf_fold_step_static(ctypes.byref(ok), storage.data_ptr(), storage.numel(), 4000, q.data_ptr(),
                                  k.data_ptr(), k.data_ptr(), 512, 4000, out.data_ptr(), None, None)
    assert rc == binding.KVF_ERR_CAPACITY                                         # 4000 + 512 > capacity
    rc = lib.kvf_fold_step_static(ctypes.byref(ok), storage.data_ptr() + 16, storage.numel(), 0, q.data_ptr(),
                                  k.data_ptr(), k.data_ptr(), 512, 0, out.data_ptr(), None, None)
    assert rc == binding.KVF_ERR_INVALID_ARG
    torch.cuda.synchronize()

"""ctypes binding of include/kvfold.h: argument marshalling only.

PyTorch appears here for device memory and streams; every step of the fold
(rotation, append, attention, split merge) runs in the library's kernels.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libkvfold.so")

KVF_OK, KVF_ERR_INVALID_ARG, KVF_ERR_CAPACITY, KVF_ERR_UNSUPPORTED, KVF_ERR_CUDA, KVF_ERR_TIMEOUT, \
    KVF_ERR_POS, KVF_ERR_RANGE = range(8)
KVF_BF16, KVF_F32 = 0, 1
KVF_ROPE_INTERLEAVED, KVF_STRICT_POS, KVF_OUT_F32, KVF_FORCE_SIMT, KVF_CACHE_INT8 = 1, 2, 4, 8, 16
KVF_HOST_UPLOAD_AHEAD, KVF_CACHE_INT4, KVF_HOST_DOWNLOAD_BEHIND, KVF_COMBINE_BEHIND = 32, 64, 128, 256

EXPORTS = [
    "kvf_cache_storage_bytes", "kvf_workspace_bytes", "kvf_cache_create", "kvf_fold_step",
    "kvf_fold_step_host", "kvf_attend", "kvf_merge_partials", "kvf_cache_len", "kvf_cache_reset", "kvf_cache_set_len", "kvf_cache_status",
    "kvf_cache_k_plane", "kvf_cache_v_plane", "kvf_cache_plan", "kvf_cache_set_splits",
    "kvf_cache_launch_count", "kvf_cache_profile", "kvf_cache_profile_read", "kvf_cache_destroy",
    "kvf_status_str", "kvf_last_cuda_error", "kvf_fold_step_static", "kvf_cache_status_word",
    "kvf_paged_pool_bytes", "kvf_paged_cache_create",
    "kvf_batch_workspace_bytes", "kvf_batch_create", "kvf_batch_fold_step", "kvf_batch_plan",
    "kvf_batch_status_word", "kvf_batch_launch_count", "kvf_batch_destroy", "kvf_cache_set_window",
    "kvf_batch_fold_step_ragged", "kvf_cache_k_scales", "kvf_cache_v_scales", "kvf_cache_sm_clock",
    "kvf_cache_host_flush", "kvf_batch_fold_step_varlen", "kvf_cache_flush",
]


class kvf_config(ctypes.Structure):
    _fields_ = [
        ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("capacity", ctypes.c_int64), ("max_chunk", ctypes.c_int32),
        ("flags", ctypes.c_uint32), ("rope_base", ctypes.c_double), ("softmax_scale", ctypes.c_double),
        ("inv_freq", ctypes.POINTER(ctypes.c_double)),
    ]


class KvfError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        lib = load()
        msg = lib.kvf_status_str(code).decode()
        if code == KVF_ERR_CUDA:
            msg += ": " + lib.kvf_last_cuda_error().decode()
        super().__init__(f"{where}: {msg}")


_lib = None


def load() -> ctypes.CDLL:
    """Load libkvfold.so; raises if the library has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2605_12471_b200.build` "
                          "(or __graft_entry__.build()) first")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, u64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64
    cfgp = ctypes.POINTER(kvf_config)
    lib.kvf_cache_storage_bytes.argtypes = [cfgp]
    lib.kvf_cache_storage_bytes.restype = ctypes.c_size_t
    lib.kvf_workspace_bytes.argtypes = [cfgp]
    lib.kvf_workspace_bytes.restype = ctypes.c_size_t
    lib.kvf_cache_create.argtypes = [cfgp, vp, ctypes.c_size_t, vp, ctypes.c_size_t, ctypes.POINTER(vp)]
    lib.kvf_cache_create.restype = ctypes.c_int
    lib.kvf_paged_pool_bytes.argtypes = [cfgp, i32]
    lib.kvf_paged_pool_bytes.restype = ctypes.c_size_t
    lib.kvf_paged_cache_create.argtypes = [cfgp, vp, ctypes.c_size_t, i32, vp, vp, ctypes.c_size_t, ctypes.POINTER(vp)]
    lib.kvf_paged_cache_create.restype = ctypes.c_int
    lib.kvf_fold_step.argtypes = [vp, vp, vp, vp, i32, i64, vp, vp, vp]
    lib.kvf_fold_step.restype = ctypes.c_int
    lib.kvf_fold_step_host.argtypes = [vp, vp, vp, vp, i32, i64, vp, vp, vp]
    lib.kvf_fold_step_host.restype = ctypes.c_int
    lib.kvf_fold_step_static.argtypes = [cfgp, vp, ctypes.c_size_t, i64, vp, vp, vp, i32, i64, vp, vp, vp]
    lib.kvf_fold_step_static.restype = ctypes.c_int
    lib.kvf_cache_host_flush.argtypes = [vp, vp]
    lib.kvf_cache_host_flush.restype = ctypes.c_int
    lib.kvf_cache_flush.argtypes = [vp, vp]
    lib.kvf_cache_flush.restype = ctypes.c_int
    lib.kvf_cache_len.argtypes = [vp]
    lib.kvf_cache_len.restype = i64
    lib.kvf_cache_reset.argtypes = [vp]
    lib.kvf_cache_reset.restype = ctypes.c_int
    lib.kvf_attend.argtypes = [vp, vp, i32, i64, vp, vp, vp]
    lib.kvf_attend.restype = ctypes.c_int
    lib.kvf_merge_partials.argtypes = [i32, i64, i32, ctypes.c_int, vp, vp, vp, vp, vp]
    lib.kvf_merge_partials.restype = ctypes.c_int
    lib.kvf_cache_set_len.argtypes = [vp, i64]
    lib.kvf_cache_set_len.restype = ctypes.c_int
    lib.kvf_cache_status.argtypes = [vp]
    lib.kvf_cache_status.restype = ctypes.c_int
    lib.kvf_cache_status_word.argtypes = [vp]
    lib.kvf_cache_status_word.restype = i32
    lib.kvf_cache_sm_clock.argtypes = [vp, ctypes.POINTER(u64)]
    lib.kvf_cache_sm_clock.restype = ctypes.c_int
    lib.kvf_cache_k_plane.argtypes = [vp]
    lib.kvf_cache_k_plane.restype = vp
    lib.kvf_cache_v_plane.argtypes = [vp]
    lib.kvf_cache_v_plane.restype = vp
    lib.kvf_cache_k_scales.argtypes = [vp]
    lib.kvf_cache_k_scales.restype = vp
    lib.kvf_cache_v_scales.argtypes = [vp]
    lib.kvf_cache_v_scales.restype = vp
    lib.kvf_cache_plan.argtypes = [vp, i32, i64, ctypes.POINTER(i32)]
    lib.kvf_cache_plan.restype = ctypes.c_int
    lib.kvf_cache_set_splits.argtypes = [vp, i32]
    lib.kvf_cache_set_splits.restype = ctypes.c_int
    lib.kvf_cache_set_window.argtypes = [vp, i32, i64]
    lib.kvf_cache_set_window.restype = ctypes.c_int
    lib.kvf_cache_launch_count.argtypes = [vp]
    lib.kvf_cache_launch_count.restype = u64
    lib.kvf_cache_profile.argtypes = [vp, i32]
    lib.kvf_cache_profile.restype = ctypes.c_int
    lib.kvf_cache_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(u64)]
    lib.kvf_cache_profile_read.restype = ctypes.c_int
    lib.kvf_cache_destroy.argtypes = [vp]
    lib.kvf_cache_destroy.restype = None
    lib.kvf_batch_workspace_bytes.argtypes = [cfgp, i32]
    lib.kvf_batch_workspace_bytes.restype = ctypes.c_size_t
    lib.kvf_batch_create.argtypes = [ctypes.POINTER(vp), i32, vp, ctypes.c_size_t, ctypes.POINTER(vp)]
    lib.kvf_batch_create.restype = ctypes.c_int
    lib.kvf_batch_fold_step.argtypes = [vp, vp, vp, vp, i32, i64, vp, vp, vp]
    lib.kvf_batch_fold_step.restype = ctypes.c_int
    lib.kvf_batch_fold_step_ragged.argtypes = [vp, vp, vp, vp, i32, ctypes.POINTER(i64), vp, vp, vp]
    lib.kvf_batch_fold_step_ragged.restype = ctypes.c_int
    lib.kvf_batch_fold_step_varlen.argtypes = [vp, vp, vp, vp, ctypes.POINTER(i32), i32, ctypes.POINTER(i64), vp, vp, vp]
    lib.kvf_batch_fold_step_varlen.restype = ctypes.c_int
    lib.kvf_batch_plan.argtypes = [vp, i32, i64, ctypes.POINTER(i32)]
    lib.kvf_batch_plan.restype = ctypes.c_int
    lib.kvf_batch_status_word.argtypes = [vp]
    lib.kvf_batch_status_word.restype = i32
    lib.kvf_batch_launch_count.argtypes = [vp]
    lib.kvf_batch_launch_count.restype = u64
    lib.kvf_batch_destroy.argtypes = [vp]
    lib.kvf_batch_destroy.restype = None
    lib.kvf_status_str.argtypes = [ctypes.c_int]
    lib.kvf_status_str.restype = ctypes.c_char_p
    lib.kvf_last_cuda_error.argtypes = []
    lib.kvf_last_cuda_error.restype = ctypes.c_char_p
    _lib = lib
    return lib


def make_config(n_q_heads: int, n_kv_heads: int, head_dim: int, dtype: str | int, capacity: int,
                max_chunk: int, rope_base: float = 10000.0, softmax_scale: float = 0.0, flags: int = 0,
                inv_freq=None) -> kvf_config:
    cfg = kvf_config()
    cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim = n_q_heads, n_kv_heads, head_dim
    cfg.dtype = {"bf16": KVF_BF16, "f32": KVF_F32}.get(dtype, dtype)
    cfg.capacity, cfg.max_chunk, cfg.flags = capacity, max_chunk, flags
    cfg.rope_base, cfg.softmax_scale = rope_base, softmax_scale
    if inv_freq is not None:
        arr = (ctypes.c_double * (head_dim // 2))(*[float(x) for x in inv_freq])
        cfg._keepalive = arr
        cfg.inv_freq = ctypes.cast(arr, ctypes.POINTER(ctypes.c_double))
    return cfg


def cache_storage_bytes(cfg: kvf_config) -> int:
    return int(load().kvf_cache_storage_bytes(ctypes.byref(cfg)))


def workspace_bytes(cfg: kvf_config) -> int:
    return int(load().kvf_workspace_bytes(ctypes.byref(cfg)))


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


class Cache:
    """One layer's accumulated K/V on the current CUDA device (kvf_cache_* calls)."""

    def __init__(self, cfg: kvf_config, device: str | torch.device = "cuda", workspace: torch.Tensor | None = None):
        lib = load()
        self.cfg = cfg
        self.device = torch.device(device)
        sb, wb = cache_storage_bytes(cfg), workspace_bytes(cfg)
        if sb == 0 or wb == 0:
            # let the library name the reason
            h = ctypes.c_void_p()
            rc = lib.kvf_cache_create(ctypes.byref(cfg), None, 0, None, 0, ctypes.byref(h))
            raise KvfError(rc if rc else KVF_ERR_INVALID_ARG, "kvf_cache_create")
        self.storage = torch.empty(sb, dtype=torch.uint8, device=self.device)
        self.workspace = workspace if workspace is not None else torch.empty(wb, dtype=torch.uint8, device=self.device)
        h = ctypes.c_void_p()
        with torch.cuda.device(self.device):
            rc = lib.kvf_cache_create(ctypes.byref(cfg), self.storage.data_ptr(), sb,
                                      self.workspace.data_ptr(), self.workspace.numel(), ctypes.byref(h))
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_cache_create")
        self._h = h
        self.torch_dtype = torch.bfloat16 if cfg.dtype == KVF_BF16 else torch.float32
        self.out_dtype = torch.float32 if (cfg.flags & KVF_OUT_F32) else self.torch_dtype

    def close(self):
        # (at interpreter shutdown the module's globals may already be gone: then the process ends anyway)
        if getattr(self, "_h", None) and load is not None:
            load().kvf_cache_destroy(self._h)
            self._h = None

    __del__ = close

    def __len__(self) -> int:
        return int(load().kvf_cache_len(self._h))

    def reset(self):
        rc = load().kvf_cache_reset(self._h)
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_cache_reset")

    def set_len(self, n: int):
        """kvf_cache_set_len: forget the rows behind row n (or resume from restored storage)."""
        rc = load().kvf_cache_set_len(self._h, int(n))
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_cache_set_len")

    def fold_step(self, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor,
                  pos0: Optional[int] = None, out: Optional[torch.Tensor] = None,
                  lse: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        """kvf_fold_step on device tensors; returns the chunk's attention output."""
        n = q.shape[0]
        for t in (q, k_new, v_new):
            assert t.is_cuda and t.is_contiguous() and t.dtype == self.torch_dtype
        if out is None:
            out = torch.empty((n, self.cfg.n_q_heads, self.cfg.head_dim), dtype=self.out_dtype, device=q.device)
        if pos0 is None:
            pos0 = len(self)
        rc = load().kvf_fold_step(self._h, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), n, int(pos0),
                                  out.data_ptr(), lse.data_ptr() if lse is not None else None,
                                  _stream_ptr(stream))
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_fold_step")
        return out

    def attend(self, q: torch.Tensor, pos0: Optional[int] = None, out: Optional[torch.Tensor] = None,
               lse: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        """kvf_attend: the queries attend to every row the cache holds; nothing is appended."""
        n = q.shape[0]
        assert q.is_cuda and q.is_contiguous() and q.dtype == self.torch_dtype
        if out is None:
            out = torch.empty((n, self.cfg.n_q_heads, self.cfg.head_dim), dtype=self.out_dtype, device=q.device)
        rc = load().kvf_attend(self._h, q.data_ptr(), n, int(len(self) if pos0 is None else pos0), out.data_ptr(),
                               lse.data_ptr() if lse is not None else None, _stream_ptr(stream))
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_attend")
        return out

    def fold_step_host(self, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, out: torch.Tensor,
                       pos0: Optional[int] = None, lse: Optional[torch.Tensor] = None,
                       stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        """kvf_fold_step_host on (pinned) host tensors; copies run on the stream."""
        n = q.shape[0]
        for t in (q, k_new, v_new, out):
            assert not t.is_cuda and t.is_contiguous()
        if pos0 is None:
            pos0 = len(self)
        rc = load().kvf_fold_step_host(self._h, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), n, int(pos0),
                                       out.data_ptr(), lse.data_ptr() if lse is not None else None,
                                       _stream_ptr(stream))
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_fold_step_host")
        return out

    def flush(self, stream: Optional[torch.cuda.Stream] = None):
        """kvf_cache_flush: the stream waits for the merge (KVF_COMBINE_BEHIND) and the result copies
        (KVF_HOST_DOWNLOAD_BEHIND) the steps so far left on the library's streams."""
        rc = load().kvf_cache_flush(self._h, _stream_ptr(stream))
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_cache_flush")

    def host_flush(self, stream: Optional[torch.cuda.Stream] = None):
        """kvf_cache_host_flush: the stream waits for the result copies of all host steps so far."""
        rc = load().kvf_cache_host_flush(self._h, _stream_ptr(stream))
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_cache_host_flush")

    def status(self) -> int:
        return int(load().kvf_cache_status(self._h))

    def status_word(self) -> int:
        """Raw device status word (0 = no bounded wait gave up; see kvf_cache_status_word)."""
        return int(load().kvf_cache_status_word(self._h))

    def sm_clock(self) -> Tuple[int, int]:
        """(SM cycles, nanoseconds) summed over one CTA (last row block, first key range) of every tensor-core attention launch so far."""
        arr = (ctypes.c_uint64 * 2)()
        rc = load().kvf_cache_sm_clock(self._h, arr)
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_cache_sm_clock")
        return int(arr[0]), int(arr[1])

    def _plane(self, ptr: int) -> torch.Tensor:
        shape = (self.cfg.n_kv_heads, self.cfg.capacity, self.cfg.head_dim)
        off = ptr - self.storage.data_ptr()
        if self.cfg.flags & KVF_CACHE_INT8:                     # int8 codes
            n = shape[0] * shape[1] * shape[2]
            return self.storage[off:off + n].view(torch.int8).view(shape)
        if self.cfg.flags & KVF_CACHE_INT4:                     # int4 codes, unpacked to int8 (a copy)
            n = shape[0] * shape[1] * shape[2] // 2
            packed = self.storage[off:off + n].view(shape[0], shape[1], shape[2] // 2).to(torch.int16)
            codes = torch.stack([packed & 15, packed >> 4], dim=-1).view(shape) - 8     # element 2i = low nibble of byte i
            return codes.to(torch.int8)
        plane_bytes = self.storage.numel() // 2
        flat = self.storage[off:off + plane_bytes].view(self.torch_dtype)
        return flat.view(shape)

    def scales(self, kv: int) -> torch.Tensor:
        """[Hkv, capacity] fp32 row scales of the K (kv = 0) or V (kv = 1) codes (KVF_CACHE_INT8 only)."""
        lib = load()
        ptr = lib.kvf_cache_v_scales(self._h) if kv else lib.kvf_cache_k_scales(self._h)
        if not ptr:
            raise ValueError("this cache holds no scales")
        off = ptr - self.storage.data_ptr()
        stride = (self.cfg.capacity + 3) // 4 * 4               # each head's scales start 16-byte aligned
        n = self.cfg.n_kv_heads * stride
        return self.storage[off:off + 4 * n].view(torch.float32).view(self.cfg.n_kv_heads, stride)[:, :self.cfg.capacity]

    def k_plane(self) -> torch.Tensor:
        """[Hkv, capacity, d] view of the rotated keys (rows >= len are not content)."""
        return self._plane(load().kvf_cache_k_plane(self._h))

    def v_plane(self) -> torch.Tensor:
        return self._plane(load().kvf_cache_v_plane(self._h))

    def plan(self, n_tokens: int, prefix_len: Optional[int] = None) -> Tuple[int, int, int, int]:
        arr = (ctypes.c_int32 * 4)()
        rc = load().kvf_cache_plan(self._h, n_tokens, len(self) if prefix_len is None else prefix_len, arr)
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_cache_plan")
        return tuple(arr)

    def set_splits(self, splits: int):
        rc = load().kvf_cache_set_splits(self._h, splits)
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_cache_set_splits")

    def set_window(self, n_sink: int, window: int):
        """Sink + window mask from the next step on (kvf_cache_set_window); (0, 0) = full prefix."""
        rc = load().kvf_cache_set_window(self._h, n_sink, window)
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_cache_set_window")

    def launch_count(self) -> int:
        return int(load().kvf_cache_launch_count(self._h))

    def profile(self, enable: bool):
        load().kvf_cache_profile(self._h, int(enable))

    def profile_read(self):
        ms = (ctypes.c_double * 3)()
        cnt = (ctypes.c_uint64 * 3)()
        rc = load().kvf_cache_profile_read(self._h, ms, cnt)
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_cache_profile_read")
        return list(ms), list(cnt)


class PagedCache(Cache):
    """A cache whose rows live in 128-token pages of a shared pool (kvf_paged_cache_create).

    `pool` is a uint8 CUDA tensor of n_pool_pages pages, `page_table` an int32 CUDA tensor with one
    pool page number per 128 tokens of capacity; both stay owned by the caller.
    """

    def __init__(self, cfg: kvf_config, pool: torch.Tensor, n_pool_pages: int, page_table: torch.Tensor,
                 workspace: torch.Tensor | None = None):
        lib = load()
        self.cfg = cfg
        self.device = pool.device
        assert page_table.dtype == torch.int32 and page_table.is_cuda and page_table.is_contiguous()
        assert page_table.numel() >= (cfg.capacity + 127) // 128
        wb = workspace_bytes(cfg)
        self.storage, self.page_table = pool, page_table
        self.workspace = workspace if workspace is not None else torch.empty(max(wb, 256), dtype=torch.uint8, device=pool.device)
        h = ctypes.c_void_p()
        with torch.cuda.device(self.device):
            rc = lib.kvf_paged_cache_create(ctypes.byref(cfg), pool.data_ptr(), pool.numel(), n_pool_pages,
                                            page_table.data_ptr(), self.workspace.data_ptr(), self.workspace.numel(),
                                            ctypes.byref(h))
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_paged_cache_create")
        self._h = h
        self.torch_dtype = torch.bfloat16
        self.out_dtype = torch.float32 if (cfg.flags & KVF_OUT_F32) else torch.bfloat16

    def k_plane(self):
        raise NotImplementedError("a paged cache has no planes; read rows through the page table")

    v_plane = k_plane

    def page_rows(self, kv: int) -> torch.Tensor:
        """[pool pages, Hkv, 128, d] view of the K (kv = 0) or V (kv = 1) blocks of the pool (bf16 pages)."""
        d, hkv = self.cfg.head_dim, self.cfg.n_kv_heads
        pages = self.storage.view(torch.bfloat16).view(-1, 2, hkv, 128, d)
        return pages[:, kv]

    def _quant_page_bytes(self) -> Tuple[int, int]:
        """(bytes of a page, bytes of one block of codes) of a quantised pool."""
        d, hkv = self.cfg.head_dim, self.cfg.n_kv_heads
        rb = d // 2 if self.cfg.flags & KVF_CACHE_INT4 else d
        return 2 * hkv * 128 * rb + 2 * hkv * 128 * 4, hkv * 128 * rb

    def page_codes(self, kv: int) -> torch.Tensor:
        """[pool pages, Hkv, 128, d] int8 codes of the K (kv = 0) or V (kv = 1) blocks of a quantised pool
        (a copy; int4 codes unpacked: element 2i is the low nibble of byte i, stored as code + 8)."""
        d, hkv = self.cfg.head_dim, self.cfg.n_kv_heads
        page, block = self._quant_page_bytes()
        raw = self.storage.view(-1, page)[:, kv * block:(kv + 1) * block]
        if self.cfg.flags & KVF_CACHE_INT4:
            packed = raw.reshape(-1, hkv, 128, d // 2).to(torch.int16)
            return (torch.stack([packed & 15, packed >> 4], dim=-1).reshape(-1, hkv, 128, d) - 8).to(torch.int8)
        return raw.reshape(-1, hkv, 128, d).view(torch.int8).clone()

    def page_scales(self, kv: int) -> torch.Tensor:
        """[pool pages, Hkv, 128] fp32 row scales of the K (kv = 0) or V (kv = 1) rows of a quantised pool (a copy)."""
        hkv = self.cfg.n_kv_heads
        page, block = self._quant_page_bytes()
        raw = self.storage.view(-1, page)[:, 2 * block + kv * hkv * 512:2 * block + (kv + 1) * hkv * 512]
        return raw.contiguous().view(torch.float32).view(-1, hkv, 128)


class Batch:
    """Paged caches of one pool that advance together (kvf_batch_* calls): one launch of each
    kernel folds one chunk into every member.  Tensors are [n_caches, n_tokens, heads, head_dim]."""

    def __init__(self, caches, workspace: torch.Tensor | None = None):
        lib = load()
        self.caches = list(caches)
        cfg = self.caches[0].cfg
        self.cfg = cfg
        wb = int(lib.kvf_batch_workspace_bytes(ctypes.byref(cfg), len(self.caches)))
        self.workspace = workspace if workspace is not None else torch.empty(max(wb, 256), dtype=torch.uint8,
                                                                             device=self.caches[0].device)
        arr = (ctypes.c_void_p * len(self.caches))(*[c._h.value for c in self.caches])
        h = ctypes.c_void_p()
        with torch.cuda.device(self.caches[0].device):
            rc = lib.kvf_batch_create(arr, len(self.caches), self.workspace.data_ptr(), self.workspace.numel(),
                                      ctypes.byref(h))
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_batch_create")
        self._h = h

    def close(self):
        if getattr(self, "_h", None) and load is not None:
            load().kvf_batch_destroy(self._h)
            self._h = None

    __del__ = close

    def fold_step(self, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, pos0=None,
                  out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                  stream: Optional[torch.cuda.Stream] = None, ragged: bool = False) -> torch.Tensor:
        """kvf_batch_fold_step, or with ragged=True kvf_batch_fold_step_ragged (members of different
        length; pos0 is then None or one position per member)."""
        assert q.dim() == 4 and q.shape[0] == len(self.caches)
        n = q.shape[1]
        for t in (q, k_new, v_new):
            assert t.is_cuda and t.is_contiguous() and t.dtype == torch.bfloat16
        if out is None:
            od = torch.float32 if (self.cfg.flags & KVF_OUT_F32) else torch.bfloat16
            out = torch.empty(q.shape, dtype=od, device=q.device)
        if ragged:
            arr = None if pos0 is None else (ctypes.c_int64 * len(self.caches))(*[int(p) for p in pos0])
            rc = load().kvf_batch_fold_step_ragged(self._h, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), n, arr,
                                                   out.data_ptr(), lse.data_ptr() if lse is not None else None,
                                                   _stream_ptr(stream))
            if rc != KVF_OK:
                raise KvfError(rc, "kvf_batch_fold_step_ragged")
            return out
        if pos0 is None:
            pos0 = len(self.caches[0])
        rc = load().kvf_batch_fold_step(self._h, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), n, int(pos0),
                                        out.data_ptr(), lse.data_ptr() if lse is not None else None,
                                        _stream_ptr(stream))
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_batch_fold_step")
        return out

    def fold_step_varlen(self, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, n_tokens, pos0=None,
                         out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                         stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        """kvf_batch_fold_step_varlen: member i folds the first n_tokens[i] rows of its block (0 = sits out)."""
        assert q.dim() == 4 and q.shape[0] == len(self.caches) == len(n_tokens)
        for t in (q, k_new, v_new):
            assert t.is_cuda and t.is_contiguous() and t.dtype == torch.bfloat16
        if out is None:
            od = torch.float32 if (self.cfg.flags & KVF_OUT_F32) else torch.bfloat16
            out = torch.empty(q.shape, dtype=od, device=q.device)
        ns = (ctypes.c_int32 * len(self.caches))(*[int(x) for x in n_tokens])
        arr = None if pos0 is None else (ctypes.c_int64 * len(self.caches))(*[int(p) for p in pos0])
        rc = load().kvf_batch_fold_step_varlen(self._h, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), ns, q.shape[1],
                                               arr, out.data_ptr(), lse.data_ptr() if lse is not None else None,
                                               _stream_ptr(stream))
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_batch_fold_step_varlen")
        return out

    def plan(self, n_tokens: int, prefix_len: Optional[int] = None) -> Tuple[int, int, int, int]:
        arr = (ctypes.c_int32 * 4)()
        rc = load().kvf_batch_plan(self._h, n_tokens, len(self.caches[0]) if prefix_len is None else prefix_len, arr)
        if rc != KVF_OK:
            raise KvfError(rc, "kvf_batch_plan")
        return tuple(arr)

    def status_word(self) -> int:
        return int(load().kvf_batch_status_word(self._h))

    def launch_count(self) -> int:
        return int(load().kvf_batch_launch_count(self._h))


def paged_pool_bytes(cfg: kvf_config, n_pages: int) -> int:
    return int(load().kvf_paged_pool_bytes(ctypes.byref(cfg), n_pages))


STATIC_SCRATCH_BYTES = 21234688


def merge_partials(parts_out: torch.Tensor, parts_lse: torch.Tensor, out: Optional[torch.Tensor] = None,
                   lse: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """kvf_merge_partials on [parts, tokens, heads, head_dim] outputs (bf16 or fp32) and [parts, tokens, heads]
    log-sum-exps; returns (out, lse)."""
    assert parts_out.is_cuda and parts_out.is_contiguous() and parts_out.dim() == 4
    assert parts_lse.is_cuda and parts_lse.is_contiguous() and parts_lse.dtype == torch.float32
    assert parts_lse.shape == parts_out.shape[:3] and parts_out.dtype in (torch.bfloat16, torch.float32)
    r, n, h, d = parts_out.shape
    if out is None:
        out = torch.empty((n, h, d), dtype=parts_out.dtype, device=parts_out.device)
    if lse is None:
        lse = torch.empty((n, h), dtype=torch.float32, device=parts_out.device)
    rc = load().kvf_merge_partials(r, n * h, d, KVF_F32 if parts_out.dtype == torch.float32 else KVF_BF16,
                                   parts_out.data_ptr(), parts_lse.data_ptr(), out.data_ptr(), lse.data_ptr(),
                                   _stream_ptr(stream))
    if rc != KVF_OK:
        raise KvfError(rc, "kvf_merge_partials")
    return out, lse


def fold_step_static(cfg: kvf_config, storage: torch.Tensor, length: int, q: torch.Tensor, k_new: torch.Tensor,
                     v_new: torch.Tensor, pos0: Optional[int] = None, out: Optional[torch.Tensor] = None,
                     lse: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """kvf_fold_step_static: the step on caller-owned planes with the library's built-in scratch.

    For callers that may not allocate device memory (a process whose memory is all in its own
    pool, a loop that must stay out of the allocator): nothing is allocated below this call when
    `out` is given.  `storage` is the uint8 tensor of the K and V planes, `length` the tokens it
    already holds; the caller adds n_tokens to its own length afterwards.
    """
    n = q.shape[0]
    for t in (q, k_new, v_new):
        assert t.is_cuda and t.is_contiguous()
    if out is None:
        od = torch.float32 if (cfg.flags & KVF_OUT_F32) or cfg.dtype == KVF_F32 else torch.bfloat16
        out = torch.empty((n, cfg.n_q_heads, cfg.head_dim), dtype=od, device=q.device)
    rc = load().kvf_fold_step_static(ctypes.byref(cfg), storage.data_ptr(), storage.numel(), int(length),
                                     q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), n,
                                     int(length if pos0 is None else pos0), out.data_ptr(),
                                     lse.data_ptr() if lse is not None else None, _stream_ptr(stream))
    if rc != KVF_OK:
        raise KvfError(rc, "kvf_fold_step_static")
    return out


def cache_for(w, capacity: Optional[int] = None, max_chunk: Optional[int] = None, flags: int = 0,
              device: str | torch.device = "cuda", workspace: torch.Tensor | None = None) -> Cache:
    """A cache shaped for a workloads.Workload."""
    cfg = make_config(w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, capacity or w.tokens,
                      max_chunk or w.chunk, rope_base=w.rope_base, flags=flags)
    return Cache(cfg, device=device, workspace=workspace)

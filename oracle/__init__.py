"""fp64 CPU oracle of the KV-Fold fold step (test infrastructure, not product).

Only tests, the smoke check and the benchmark's CPU-baseline legs may import
this package.  It builds ``kvfold_oracle.c`` with gcc into a shared object next
to the source and wraps it with ctypes and numpy; it imports nothing from the
CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kvfold_oracle.c")
_LIB = os.path.join(_HERE, "libkvfold_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (gcc, OpenMP across independent rows, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
             "-shared", "-fPIC", _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    dp = ctypes.POINTER(ctypes.c_double)
    fp = ctypes.POINTER(ctypes.c_float)
    ip = ctypes.POINTER(ctypes.c_int32)
    lib.okvf_inv_freq.argtypes = [ctypes.c_double, ctypes.c_int, dp]
    lib.okvf_inv_freq.restype = None
    lib.okvf_cache_create.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int64,
                                      ctypes.c_double, ctypes.c_double, ctypes.c_int, dp]
    lib.okvf_cache_create.restype = ctypes.c_void_p
    lib.okvf_cache_destroy.argtypes = [ctypes.c_void_p]
    lib.okvf_cache_destroy.restype = None
    lib.okvf_cache_len.argtypes = [ctypes.c_void_p]
    lib.okvf_cache_len.restype = ctypes.c_int64
    lib.okvf_cache_reset.argtypes = [ctypes.c_void_p]
    lib.okvf_cache_reset.restype = None
    lib.okvf_cache_set_quant.argtypes = [ctypes.c_void_p, ctypes.c_int]
    lib.okvf_cache_set_quant.restype = ctypes.c_int
    lib.okvf_quant_row.argtypes = [fp, ctypes.c_int, ctypes.c_int, ip, fp, fp]
    lib.okvf_quant_row.restype = None
    lib.okvf_cache_set_window.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64]
    lib.okvf_cache_set_window.restype = None
    lib.okvf_cache_k.argtypes = [ctypes.c_void_p]
    lib.okvf_cache_k.restype = dp
    lib.okvf_cache_v.argtypes = [ctypes.c_void_p]
    lib.okvf_cache_v.restype = dp
    lib.okvf_cache_bytes.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int64, ctypes.c_int]
    lib.okvf_cache_bytes.restype = ctypes.c_int64
    lib.okvf_rope_fp64.argtypes = [dp, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int64,
                                   dp, ctypes.c_int, dp]
    lib.okvf_rope_fp64.restype = None
    lib.okvf_rope_faithful.argtypes = [fp, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                       ctypes.c_int64, dp, ctypes.c_int, ctypes.c_int, fp]
    lib.okvf_rope_faithful.restype = None
    lib.okvf_fold_step.argtypes = [ctypes.c_void_p, dp, dp, dp, ctypes.c_int64, ctypes.c_int64,
                                   ip, ctypes.c_int64, dp, dp, dp]
    lib.okvf_fold_step.restype = ctypes.c_int
    _lib = lib
    return lib


def _dptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def inv_freq(rope_base: float, head_dim: int) -> np.ndarray:
    out = np.empty(head_dim // 2, dtype=np.float64)
    _load().okvf_inv_freq(float(rope_base), int(head_dim), _dptr(out))
    return out


def cache_bytes(n_kv_heads: int, head_dim: int, tokens: int, elem_bytes: int) -> int:
    return int(_load().okvf_cache_bytes(n_kv_heads, head_dim, tokens, elem_bytes))


def rope_fp64(x, pos0: int, inv_freq_table, interleaved: bool = False) -> np.ndarray:
    """x: [n, heads, d]; token i rotated at position pos0 + i (fp64)."""
    x = _f64(x)
    n, heads, d = x.shape
    y = np.empty_like(x)
    t = _f64(inv_freq_table)
    _load().okvf_rope_fp64(_dptr(x), n, heads, d, int(pos0), _dptr(t), int(interleaved), _dptr(y))
    return y


def rope_faithful(x, pos0: int, inv_freq_table, interleaved: bool = False,
                  to_bf16: bool = False) -> np.ndarray:
    """fp32 (optionally bf16-rounded) rotation with the cache's exact operation order."""
    x = np.ascontiguousarray(np.asarray(x, dtype=np.float32))
    n, heads, d = x.shape
    y = np.empty_like(x)
    t = _f64(inv_freq_table)
    fp = ctypes.POINTER(ctypes.c_float)
    _load().okvf_rope_faithful(x.ctypes.data_as(fp), n, heads, d, int(pos0), _dptr(t),
                               int(interleaved), int(to_bf16), y.ctypes.data_as(fp))
    return y


def quant_rows_int8(x):
    return quant_rows(x, 8)


def quant_rows(x, bits: int):
    """Round trip of the rows of x [..., d] (fp32) through int8 or int4 codes:
    (codes int32, scales fp32 [...], stored fp32)."""
    x = np.ascontiguousarray(np.asarray(x, dtype=np.float32))
    d = x.shape[-1]
    flat = x.reshape(-1, d)
    codes = np.empty(flat.shape, dtype=np.int32)
    scales = np.empty(flat.shape[0], dtype=np.float32)
    stored = np.empty_like(flat)
    fp = ctypes.POINTER(ctypes.c_float)
    ip = ctypes.POINTER(ctypes.c_int32)
    lib = _load()
    for r in range(flat.shape[0]):
        sc = ctypes.c_float()
        lib.okvf_quant_row(flat[r].ctypes.data_as(fp), d, int(bits), codes[r].ctypes.data_as(ip), ctypes.byref(sc),
                           stored[r].ctypes.data_as(fp))
        scales[r] = sc.value
    return codes.reshape(x.shape), scales.reshape(x.shape[:-1]), stored.reshape(x.shape)


class OracleCache:
    """One layer's accumulated K/V in fp64 plus the fold step on it."""

    def __init__(self, n_q_heads: int, n_kv_heads: int, head_dim: int, capacity: int,
                 rope_base: float = 10000.0, softmax_scale: float = 0.0,
                 interleaved: bool = False, inv_freq_table=None):
        lib = _load()
        self.H, self.Hkv, self.d, self.capacity = n_q_heads, n_kv_heads, head_dim, capacity
        tab = None
        if inv_freq_table is not None:
            self._tab = _f64(inv_freq_table)
            tab = _dptr(self._tab)
        self._h = lib.okvf_cache_create(n_q_heads, n_kv_heads, head_dim, capacity,
                                        float(rope_base), float(softmax_scale), int(interleaved),
                                        tab)
        if not self._h:
            raise ValueError("okvf_cache_create rejected the configuration")

    def close(self):
        if getattr(self, "_h", None):
            _load().okvf_cache_destroy(self._h)
            self._h = None

    __del__ = close

    def __len__(self) -> int:
        return int(_load().okvf_cache_len(self._h))

    def reset(self):
        _load().okvf_cache_reset(self._h)

    def set_quant(self, bits: int):
        """Quantised storage: rows go through an int8 / int4 round trip when appended (bits = 8 / 4; 0 = off)."""
        if _load().okvf_cache_set_quant(self._h, int(bits)) != 0:
            raise ValueError("only 0, 8 or 4 bits")

    def set_window(self, n_sink: int, window: int):
        """Sink + window variant: earlier chunks' rows are visible only if among the first n_sink
        or the last `window` before the chunk (window <= 0: all of them)."""
        _load().okvf_cache_set_window(self._h, int(n_sink), int(window))

    def _plane(self, ptr) -> np.ndarray:
        a = np.ctypeslib.as_array(ptr, shape=(self.Hkv, self.capacity, self.d))
        return a[:, :len(self), :]

    def k(self) -> np.ndarray:
        """Rotated keys held so far, [Hkv, len, d] (a view)."""
        return self._plane(_load().okvf_cache_k(self._h))

    def v(self) -> np.ndarray:
        return self._plane(_load().okvf_cache_v(self._h))

    def fold_step(self, q, k_new, v_new, pos0: Optional[int] = None,
                  rows: Optional[Sequence[int]] = None, want_stats: bool = False):
        """Append the chunk and return its attention output [n_out, H, d] (fp64).

        pos0 defaults to the current length (positions continue across chunks).
        """
        q, k_new, v_new = _f64(q), _f64(k_new), _f64(v_new)
        n = q.shape[0]
        assert q.shape == (n, self.H, self.d), q.shape
        assert k_new.shape == (n, self.Hkv, self.d) and v_new.shape == (n, self.Hkv, self.d)
        if pos0 is None:
            pos0 = len(self)
        rows_arr, rows_ptr, n_rows = None, None, 0
        if rows is not None:
            rows_arr = np.ascontiguousarray(np.asarray(rows, dtype=np.int32))
            n_rows = rows_arr.shape[0]
            if n_rows == 0:           # append only: keep the pointer non-null
                rows_arr = np.zeros(1, dtype=np.int32)
            rows_ptr = rows_arr.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
        n_out = n_rows if rows is not None else n
        out = np.empty((n_out, self.H, self.d), dtype=np.float64)
        lse = np.empty((n_out, self.H), dtype=np.float64)
        rowsum = np.empty((n_out, self.H), dtype=np.float64)
        rc = _load().okvf_fold_step(self._h, _dptr(q), _dptr(k_new), _dptr(v_new), n, int(pos0),
                                    rows_ptr, n_rows, _dptr(out), _dptr(lse), _dptr(rowsum))
        if rc == 2:
            raise OverflowError("oracle cache capacity exceeded")
        if rc != 0:
            raise ValueError(f"okvf_fold_step failed with code {rc}")
        if want_stats:
            return out, lse, rowsum
        return out

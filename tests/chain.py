"""Test helper: drive the CUDA cache and the fp64 oracle through the same chain of chunks.

Inputs are drawn once (workloads.chunk_inputs) and the oracle receives the very bits the GPU
got, widened to fp64, so input rounding is never counted as error.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, Iterable, List, Optional, Sequence

import numpy as np
import torch

import oracle
from paper_2605_12471_b200 import binding, workloads

# Tolerances of the fold step against the fp64 oracle (max abs / mean abs).
TOL = {"f32": (1e-5, 1e-5), "bf16": (2e-2, 5e-3)}


@dataclasses.dataclass
class ChainResult:
    max_abs: float = 0.0
    sum_abs: float = 0.0
    count: int = 0
    sum_sq_err: float = 0.0
    sum_sq_ref: float = 0.0
    per_step: Dict[int, float] = dataclasses.field(default_factory=dict)
    lse_max_abs: float = 0.0

    @property
    def mean_abs(self) -> float:
        return self.sum_abs / max(self.count, 1)

    @property
    def rel_rms(self) -> float:
        return float(np.sqrt(self.sum_sq_err / max(self.sum_sq_ref, 1e-300)))

    def add(self, step: int, got: np.ndarray, ref: np.ndarray):
        err = np.abs(got.astype(np.float64) - ref)
        m = float(err.max()) if err.size else 0.0
        self.max_abs = max(self.max_abs, m)
        self.per_step[step] = max(self.per_step.get(step, 0.0), m)
        self.sum_abs += float(err.sum())
        self.count += err.size
        self.sum_sq_err += float((err ** 2).sum())
        self.sum_sq_ref += float((ref ** 2).sum())


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


def sample_rows(n: int, rng: np.random.Generator, extra: int = 4) -> List[int]:
    fixed = {0, 1, n // 2 - 1, n // 2, n - 2, n - 1}
    rows = {r for r in fixed if 0 <= r < n}
    if n > len(rows):
        rows.update(int(x) for x in rng.integers(0, n, size=extra))
    return sorted(rows)


def run_chain(w: workloads.Workload, chunks: Sequence[int], seed: int = 0, flags: int = 0,
              check_steps: Optional[Iterable[int]] = None, rows_per_step: Optional[int] = None,
              splits: int = 0, cache: Optional[binding.Cache] = None, check_lse: bool = True,
              keep_outputs: bool = False, positions: Optional[Sequence[int]] = None):
    """Fold `chunks` (a list of chunk lengths) on the GPU and in the oracle.

    check_steps: steps whose outputs are compared (None = all).  rows_per_step: None compares
    every row of a checked step, otherwise a fixed + seeded-random sample of rows.
    Returns (ChainResult, cache, oracle_cache, outputs or None).
    """
    total = int(sum(chunks))
    own = cache is None
    if own:
        cache = binding.cache_for(w, capacity=total, max_chunk=max(chunks), flags=flags)
    if splits:
        cache.set_splits(splits)
    oc = oracle.OracleCache(w.n_q_heads, w.n_kv_heads, w.head_dim, total, rope_base=w.rope_base,
                            interleaved=bool(flags & binding.KVF_ROPE_INTERLEAVED))
    check = None if check_steps is None else set(check_steps)
    rng = np.random.default_rng(seed + 12345)
    res = ChainResult()
    outs = [] if keep_outputs else None
    for t, n in enumerate(chunks):
        q, k, v = workloads.chunk_inputs(w, seed, t, device="cuda", n_tokens=n)
        pos0 = len(cache) if positions is None else positions[t]
        lse = torch.empty((n, w.n_q_heads), dtype=torch.float32, device="cuda") if check_lse else None
        out = cache.fold_step(q, k, v, pos0=pos0, lse=lse)
        if keep_outputs:
            outs.append(out.clone())
        checked = check is None or t in check
        rows = None
        if checked and rows_per_step is not None:
            rows = sample_rows(n, rng, rows_per_step)
        elif not checked:
            rows = []
        if rows is not None and len(rows) == 0:
            oc.fold_step(to_f64(q), to_f64(k), to_f64(v), pos0=pos0, rows=[])    # append only
            continue
        ref, ref_lse, _ = oc.fold_step(to_f64(q), to_f64(k), to_f64(v), pos0=pos0, rows=rows, want_stats=True)
        got = out if rows is None else out[rows]
        res.add(t, to_f64(got), ref)
        if check_lse:
            got_lse = to_f64(lse if rows is None else lse[rows])
            res.lse_max_abs = max(res.lse_max_abs, float(np.abs(got_lse - ref_lse).max()))
        assert len(cache) == len(oc)
    torch.cuda.synchronize()
    assert cache.status() == binding.KVF_OK, hex(cache.status_word())
    return res, cache, oc, outs


def assert_within(res: ChainResult, dtype: str, what: str = ""):
    mx, mean = TOL[dtype]
    assert res.count > 0
    assert res.max_abs <= mx, f"{what}: max abs {res.max_abs:.3e} > {mx} (per step {res.per_step})"
    assert res.mean_abs <= mean, f"{what}: mean abs {res.mean_abs:.3e} > {mean}"


# ------------------------------------------------------------------ cache contents, bit for bit
def cache_rows(cache, kv: int, start: int, n: int, table: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Rows [start, start + n) of the K (kv = 0) or V (kv = 1) side of a cache as [Hkv, n, d]:
    a slice of the plane, or for a paged cache the rows its page table names."""
    if table is None:
        plane = cache.v_plane() if kv else cache.k_plane()
        return plane[:, start:start + n]
    assert start % 128 == 0
    pages = cache.page_rows(kv)[table[start // 128:(start + n + 127) // 128].long()]   # [pages, Hkv, 128, d]
    rows = pages.permute(1, 0, 2, 3).reshape(pages.shape[1], -1, pages.shape[3])
    return rows[:, :n]


def ulp_distance(a: torch.Tensor, b: torch.Tensor) -> torch.Tensor:
    """Distance in units of the last place between two bf16 or fp32 tensors of finite values."""
    if a.dtype == torch.bfloat16:
        ia, ib = a.view(torch.int16).to(torch.int64), b.view(torch.int16).to(torch.int64)
        mag = 0x7FFF
    else:
        ia, ib = a.view(torch.int32).to(torch.int64), b.view(torch.int32).to(torch.int64)
        mag = 0x7FFFFFFF
    ia = torch.where(ia < 0, -(ia & mag), ia)          # sign-magnitude -> monotone integers
    ib = torch.where(ib < 0, -(ib & mag), ib)
    return (ia - ib).abs()


class CacheBits:
    """Accumulates the comparison of appended rows with what the paper's append must have left:
    V rows verbatim, K rows equal to the oracle's rotation in the cache dtype and operation order
    (contract: at most 1 ulp apart, and at most 1e-5 of all elements different at all, because the
    device's and the host's fp64 cos/sin may differ in their last bit)."""

    def __init__(self):
        self.elements = 0
        self.differing = 0
        self.max_ulp = 0
        self.v_equal = True

    def add(self, cache, w: workloads.Workload, k: torch.Tensor, v: torch.Tensor, start: int, pos0: int,
            interleaved: bool = False, table: Optional[torch.Tensor] = None):
        n = k.shape[0]
        tab = oracle.inv_freq(w.rope_base, w.head_dim)
        want = oracle.rope_faithful(k.float().cpu().numpy(), pos0, tab, interleaved=interleaved,
                                    to_bf16=(w.dtype == "bf16"))
        want = torch.from_numpy(want).to(k.dtype).permute(1, 0, 2).contiguous().to(k.device)     # [Hkv, n, d]
        dist = ulp_distance(cache_rows(cache, 0, start, n, table).contiguous(), want)
        self.elements += dist.numel()
        self.differing += int((dist != 0).sum())
        self.max_ulp = max(self.max_ulp, int(dist.max()))
        got_v = cache_rows(cache, 1, start, n, table).contiguous()
        self.v_equal = self.v_equal and bool(torch.equal(got_v.view(torch.uint8),
                                                         v.permute(1, 0, 2).contiguous().view(torch.uint8)))

    def check(self, what: str = ""):
        assert self.elements > 0
        assert self.v_equal, f"{what}: value rows are not the inputs verbatim"
        assert self.max_ulp <= 1, f"{what}: a key element is {self.max_ulp} ulp from the oracle's rotation"
        assert self.differing <= 1e-5 * self.elements, f"{what}: {self.differing} of {self.elements} key elements differ"


def assert_chain_cache_bits(cache, w: workloads.Workload, chunks: Sequence[int], seed: int, flags: int = 0,
                            positions: Optional[Sequence[int]] = None, what: str = ""):
    """Every row a chain of run_chain(w, chunks, seed) appended, compared in full (the chunks'
    inputs are drawn again from their seeds)."""
    bits = CacheBits()
    start = 0
    for t, n in enumerate(chunks):
        _, k, v = workloads.chunk_inputs(w, seed, t, device="cuda", n_tokens=n)
        bits.add(cache, w, k, v, start, start if positions is None else positions[t],
                 interleaved=bool(flags & binding.KVF_ROPE_INTERLEAVED))
        start += n
    bits.check(what)
    return bits

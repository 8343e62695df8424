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

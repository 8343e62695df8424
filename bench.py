#!/usr/bin/env python
"""Benchmark of the KV-Fold fold step on B200.

One benchmark "step" is one whole chain of the deep-chain workload: the cache is reset to the
empty accumulator and 131 072 tokens are folded in 512 chunks of 256 (chain depth 511), every
chunk going through rotate+append, prefix+chunk attention and (when split) the combine kernel.
`value` is tokens folded per second with the inputs resident in HBM; `e2e` is the same chain
through the host-buffer entry point (pinned host q/k/v in, out back, copies inside the timing).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank folds its own
independent sequence: there is no exchange on the data path, the only collective is the
max-over-ranks of the elapsed time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2605_12471_b200 import workloads  # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# DRAM bytes (read + write) of one attention launch per algorithmic cache byte it reads, from an
# ncu capture of the last steps of a 65 536-token chain of 256-token chunks (too large to capture
# at 131 072 tokens; traffic grows in proportion to the cache rows read, so the ratio carries
# over).  Set to None whenever the attention kernel changes after the capture.
NCU_TRAFFIC_BYTES_PER_CACHE_BYTE = 1.033
NCU_TRAFFIC_SOURCE = ("ncu capture (dram__bytes_read.sum + dram__bytes_write.sum) of the attention kernel on the "
                      "last steps of a 65 536-token chain of 256-token chunks: 1.033 DRAM bytes per algorithmic "
                      "cache byte, scaled by the cache rows a launch of this run reads")
NOMINAL = {"bf16_tflops": 2250.0, "hbm_gbs": 7700.0}      # dense bf16 and HBM3e figures of the B200 data sheet
TENSOR_FLOP_PER_SM_CLOCK = 8192.0                         # one 128 x 128 x 16 bf16 MMA (524 288 FLOP) per 64 clocks
N_SMS = 148


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.proc, self.lines = gpu_index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()          # the exact process started above
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower() == "active":
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


class NvmlClock:
    """Reads the SM clock of one GPU through NVML about once a millisecond (a read, nothing is set),
    with host timestamps, so that short stretches of a run can be given their own median clock."""

    def __init__(self, gpu_index: int):
        self.samples, self._stop, self.thread, self.handle = [], threading.Event(), None, None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(gpu_index)
        except Exception:            # no NVML: the per-bin clocks are simply left out
            self.handle = None

    def start(self):
        if self.handle is None:
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        while not self._stop.is_set():
            try:
                mhz = self.nv.nvmlDeviceGetClockInfo(self.handle, self.nv.NVML_CLOCK_SM)
            except Exception:
                return
            self.samples.append((time.perf_counter(), float(mhz)))
            time.sleep(0.001)

    def stop(self):
        self._stop.set()
        if self.thread is not None:
            self.thread.join(timeout=2)

    def median_between(self, t0: float, t1: float):
        xs = [m for t, m in self.samples if t0 <= t <= t1]
        return statistics.median(xs) if xs else None


def set_oracle_threads(n: int) -> bool:
    """Thread count of the oracle's OpenMP runtime (the oracle itself is left as it stands)."""
    import ctypes
    try:
        ctypes.CDLL("libgomp.so.1").omp_set_num_threads(int(n))
        return True
    except OSError:
        return False


def oracle_rate(w: workloads.Workload, seed: int, rows_per_step: int, repeats: int, prefix: int):
    """Times the fp64 oracle (as it stands) on `rows_per_step` query rows of the chunk that follows
    `prefix` cached tokens.  Returns (visible (query,key) pairs per second, seconds per repeat,
    threads)."""
    import numpy as np

    import oracle
    oc = oracle.OracleCache(w.n_q_heads, w.n_kv_heads, w.head_dim, prefix + w.chunk * (repeats + 1),
                            rope_base=w.rope_base)
    gen = np.random.default_rng(seed)
    block = 8192
    done = 0
    while done < prefix:                                   # fill the accumulator (not timed)
        n = min(block, prefix - done)
        k = gen.standard_normal((n, w.n_kv_heads, w.head_dim))
        v = gen.standard_normal((n, w.n_kv_heads, w.head_dim))
        q = np.zeros((n, w.n_q_heads, w.head_dim))
        oc.fold_step(q, k, v, rows=[])
        done += n
    rows = sorted(set(int(x) for x in np.linspace(0, w.chunk - 1, rows_per_step)))
    times, pairs = [], 0
    for _ in range(repeats):
        q = gen.standard_normal((w.chunk, w.n_q_heads, w.head_dim))
        k = gen.standard_normal((w.chunk, w.n_kv_heads, w.head_dim))
        v = gen.standard_normal((w.chunk, w.n_kv_heads, w.head_dim))
        p0 = len(oc)
        t0 = time.perf_counter()
        oc.fold_step(q, k, v, rows=rows)
        times.append(time.perf_counter() - t0)
        pairs = sum(p0 + r + 1 for r in rows)
    threads = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
    return pairs / statistics.median(times), times, threads, rows


def tokens_per_s_from_pairs(w: workloads.Workload, pairs_per_s: float, prefill: int = 0) -> float:
    """Tokens prefill .. T-1 see (T(T+1) - P(P+1))/2 (query, key) pairs: tokens/s = pairs/s x tokens / pairs."""
    t, p0 = w.tokens, prefill
    return pairs_per_s * (t - p0) / ((t * (t + 1) - p0 * (p0 + 1)) / 2.0)


def run_reference(args, w):
    """The reference arm: the CPU oracle, on a bounded sample of the same workload per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    prefix = w.tokens - w.chunk
    import numpy as np

    import oracle
    oc = oracle.OracleCache(w.n_q_heads, w.n_kv_heads, w.head_dim, w.tokens + w.chunk * (args.steps + args.warmup),
                            rope_base=w.rope_base)
    gen = np.random.default_rng(args.seed)
    done = 0
    while done < prefix:
        n = min(8192, prefix - done)
        oc.fold_step(np.zeros((n, w.n_q_heads, w.head_dim)), gen.standard_normal((n, w.n_kv_heads, w.head_dim)),
                     gen.standard_normal((n, w.n_kv_heads, w.head_dim)), rows=[])
        done += n
    rows = sorted(set(int(x) for x in np.linspace(0, w.chunk - 1, args.ref_rows)))
    elapsed, pairs = 0.0, 0
    for it in range(args.warmup + args.steps):
        q = gen.standard_normal((w.chunk, w.n_q_heads, w.head_dim))
        k = gen.standard_normal((w.chunk, w.n_kv_heads, w.head_dim))
        v = gen.standard_normal((w.chunk, w.n_kv_heads, w.head_dim))
        p0 = len(oc)
        t0 = time.perf_counter()
        oc.fold_step(q, k, v, rows=rows)
        dt = time.perf_counter() - t0
        if it >= args.warmup:
            elapsed += dt
            pairs += sum(p0 + r + 1 for r in rows)
    value = tokens_per_s_from_pairs(w, pairs / elapsed, args.prefill)
    threads = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
    sample = (f"{len(rows)} query rows x {w.n_q_heads} heads per step at prefix >= {prefix} (last chunk of the "
              f"chain), fp64 oracle; tokens/s extrapolated linearly in visible (query,key) pairs")
    line = {
        "impl": "reference", "metric": "fold-step tokens/s", "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * elapsed / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "tokens": w.tokens, "chunk": w.chunk, "prefill": args.prefill,
                   "fold_steps_per_step": (w.tokens - args.prefill) // w.chunk, "n_q_heads": w.n_q_heads,
                   "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "rope_base": w.rope_base},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def run_full_stack(args):
    """Memory-scale fold (not the headline line): `--sequences` independent sequences x `--layers`
    layers, each layer its own bf16 cache, 131 072 tokens per sequence in chunks of 1024; per chunk
    all layers' fold steps are issued on one stream.  Every (sequence, layer) draws its chunk
    inputs once from its own seed and reuses them for every chunk: values do not change the work,
    and 16 384 fresh draws would not fit beside 64 GiB of cache."""
    from paper_2605_12471_b200 import binding
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the fold step has no CPU path")
    torch.cuda.set_device(0)
    w = workloads.FULL_STACK.with_(n_sequences=args.sequences, n_layers=args.layers, tokens=args.tokens or 131072)
    C, T, N = w.chunk, w.tokens, w.n_steps
    cfg = binding.make_config(w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, T, C, rope_base=w.rope_base)
    ws = torch.empty(binding.workspace_bytes(cfg), dtype=torch.uint8, device="cuda")     # one workspace, one stream
    caches, inputs = [], []
    lib, stream = binding.load(), torch.cuda.current_stream().cuda_stream
    keys = [(sq, ly) for sq in range(w.n_sequences) for ly in range(w.n_layers)]
    for sq, ly in keys:
        inputs.append(workloads.chunk_inputs(w, args.seed, 0, sequence=sq, layer=ly, device="cuda"))
    if args.batched:
        # every cache in 128-token pages of one pool (tables dealt from one shuffled deck); a chunk is ONE
        # step of the batch: one launch of each kernel for all caches
        per = (T + 127) // 128
        n_pool = len(keys) * per
        deck = torch.randperm(n_pool, generator=torch.Generator().manual_seed(args.seed)).to(torch.int32)
        tables = deck.view(len(keys), per).cuda()
        pool = torch.empty(binding.paged_pool_bytes(cfg, n_pool), dtype=torch.uint8, device="cuda")
        caches = [binding.PagedCache(cfg, pool, n_pool, tables[i], workspace=ws) for i in range(len(keys))]
        batch = binding.Batch(caches)
        bq, bk, bv = (torch.stack([x[j] for x in inputs]).contiguous() for j in range(3))
        inputs = None
        bout = torch.empty_like(bq)
        bh = batch._h

        def chain():
            for c in caches:
                c.reset()
            for t in range(N):
                rc = lib.kvf_batch_fold_step(bh, bq.data_ptr(), bk.data_ptr(), bv.data_ptr(), C, t * C, bout.data_ptr(), None, stream)
                if rc:
                    raise binding.KvfError(rc, "kvf_batch_fold_step")
    else:
        caches = [binding.Cache(cfg, workspace=ws) for _ in keys]
        out = torch.empty_like(inputs[0][0])
        ptrs = [(c._h, q.data_ptr(), k.data_ptr(), v.data_ptr()) for c, (q, k, v) in zip(caches, inputs)]

        def chain():
            for c in caches:
                c.reset()
            for t in range(N):
                for h, qp, kp, vp in ptrs:
                    rc = lib.kvf_fold_step(h, qp, kp, vp, C, t * C, out.data_ptr(), None, stream)
                    if rc:
                        raise binding.KvfError(rc, "kvf_fold_step")

    sampler = ClockSampler(0)
    chain()                                               # warm-up pass
    torch.cuda.synchronize()
    sampler.start()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    chain()
    b.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = a.elapsed_time(b)
    assert all(len(c) == T for c in caches) and all(c.status() == binding.KVF_OK for c in caches)
    assert not args.batched or batch.status_word() == 0
    ncache = len(caches)
    flops = ncache * w.flops_chain()
    pk = peaks()
    line = {"metric": "fold-step tokens/s", "value": ncache * T / (ms * 1e-3), "unit": "tokens/s (layer-tokens)", "n_gpus": 1,
            "steps": 1, "warmup": 1, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": w.dtype, "data": "synthetic",
            "config": {"workload": w.name, "sequences": w.n_sequences, "layers": w.n_layers, "tokens": T, "chunk": C,
                       "caches": ncache, "cache_gib": ncache * binding.cache_storage_bytes(cfg) / 2 ** 30,
                       "fold_steps": ncache * N, "l2": "inputs larger than L2",
                       "launch": "one batch step per chunk (one launch of each kernel for all caches, paged pool)"
                                 if args.batched else "one fold step per cache and chunk"},
            "attention_tflops_whole_step": flops / (ms * 1e-3) / 1e12,
            "frac_of_sustained_bf16_peak": flops / (ms * 1e-3) / 1e12 / pk["bf16_tflops_sustained"],
            "gpu_launches": (batch.launch_count() if args.batched else sum(c.launch_count() for c in caches)) // 2,
            "clocks": clocks}
    print(json.dumps(line), flush=True)


def run_batch_decode(args):
    """Sequences decoded together (not the headline line): `--caches` paged caches of one pool, each holding
    `--prefill` tokens (folded in lock step, 2048 at a time, outside the timed region), then `--steps` timed
    batch steps of `--chunk` tokens per member (default one), every member with inputs of its own.  The step is
    bound by the cache read: value = tokens/s over all members, roofline = cache bytes read per second."""
    from paper_2605_12471_b200 import binding
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the fold step has no CPU path")
    torch.cuda.set_device(0)
    B, P, n = args.caches, args.prefill or 16384, args.chunk or 1
    if P % 2048:
        raise SystemExit("--prefill must be a multiple of 2048")
    w = workloads.DEEP_CHAIN
    H, Hkv, d = w.n_q_heads, w.n_kv_heads, w.head_dim
    steps = max(args.steps, 1) * 400                             # a timed stretch of about half a second
    cap = P + (args.warmup + 1) * steps * n + 128
    flags = binding.KVF_CACHE_INT8 if args.cache_int8 else binding.KVF_CACHE_INT4 if args.cache_int4 else 0
    cfg = binding.make_config(H, Hkv, d, "bf16", cap, 2048, rope_base=w.rope_base, flags=flags)
    per = (cap + 127) // 128
    n_pool = B * per
    deck = torch.randperm(n_pool, generator=torch.Generator().manual_seed(args.seed)).to(torch.int32)
    tables = deck.view(B, per).cuda()
    pool = torch.zeros(binding.paged_pool_bytes(cfg, n_pool), dtype=torch.uint8, device="cuda")
    ws = torch.empty(binding.workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    caches = [binding.PagedCache(cfg, pool, n_pool, tables[i], workspace=ws) for i in range(B)]
    batch = binding.Batch(caches)
    gen = torch.Generator(device="cuda").manual_seed(args.seed)

    def draw(tokens, heads):
        return torch.randn((B, tokens, heads, d), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)

    fq, fk, fv = draw(2048, H), draw(2048, Hkv), draw(2048, Hkv)
    for _ in range(P // 2048):
        batch.fold_step(fq, fk, fv)
    del fq, fk, fv
    q, k, v = draw(n, H), draw(n, Hkv), draw(n, Hkv)
    out = torch.empty_like(q)
    lib, bh, stream = binding.load(), batch._h, torch.cuda.current_stream().cuda_stream

    def run(count):
        for _ in range(count):
            rc = lib.kvf_batch_fold_step(bh, q.data_ptr(), k.data_ptr(), v.data_ptr(), n, len(caches[0]), out.data_ptr(),
                                         None, stream)
            if rc:
                raise binding.KvfError(rc, "kvf_batch_fold_step")

    for _ in range(max(args.warmup, 1)):
        run(steps)
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    first = len(caches[0])
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    run(steps)
    b.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = a.elapsed_time(b)
    assert batch.status_word() == 0 and all(c.status() == binding.KVF_OK for c in caches)
    row_bytes = 2 * Hkv * ((d + 4) if args.cache_int8 else (d // 2 + 4) if args.cache_int4 else 2 * d)
    mean_rows = first + (steps * n + n) / 2.0                    # rows a step reads per cache, averaged over the stretch
    gbs = B * mean_rows * row_bytes * steps / (ms * 1e-3) / 1e9
    pk = peaks()
    line = {"metric": "fold-step tokens/s", "value": B * n * steps / (ms * 1e-3), "unit": "tokens/s", "n_gpus": 1,
            "steps": steps, "warmup": max(args.warmup, 1), "ms_per_step": ms / steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "batch_decode", "caches": B, "prefix": first, "tokens_per_member": n,
                       "n_q_heads": H, "n_kv_heads": Hkv, "head_dim": d,
                       "cache_storage": "int8 codes + fp32 row scales" if args.cache_int8 else
                                        "int4 codes + fp32 row scales" if args.cache_int4 else "bf16 rows",
                       "paged": True, "plan": dict(zip(("tensor_core", "splits", "ctas", "kernels"), batch.plan(n))),
                       "launch": "one batch step per token (one launch of each kernel for all caches)",
                       "l2": "inputs larger than L2 (%.2f GB of cache rows per step)" % (B * mean_rows * row_bytes / 1e9)},
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": gbs / pk["hbm_gbs"],
                         "peak_source": "measured copy bandwidth" if pk["_source"] == "measured" else "fallback copy bandwidth", "traffic": None,
                         "kernel": "whole step (rotate + append, attention, merge)",
                         "cache_bytes_per_step": B * mean_rows * row_bytes},
            "cpu_baseline": None, "e2e": None, "gpu_launches": batch.launch_count(), "clocks": clocks}
    print(json.dumps(line), flush=True)


def run_multi_needle(args):
    """Several questions about one folded haystack (not the headline line).  The paper's multi-needle protocol
    queries K keys separately on the same context: the haystack (`--prefill` tokens, default 129 024) is folded
    ONCE, outside the timed region; the timed region is `--needles` questions, each a question chunk of `--chunk`
    tokens (default 32) and 30 tokens decoded one at a time, after which kvf_cache_set_len takes the cache back to
    the haystack.  Every step is bound by the cache read; value = tokens folded per second in the timed region."""
    from paper_2605_12471_b200 import binding
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the fold step has no CPU path")
    torch.cuda.set_device(0)
    w = workloads.DEEP_CHAIN
    H, Hkv, d = w.n_q_heads, w.n_kv_heads, w.head_dim
    P, nq, ndec, K = args.prefill or 129024, args.chunk or 32, 30, args.needles
    if P % 2048:
        raise SystemExit("--prefill must be a multiple of 2048")
    flags = binding.KVF_CACHE_INT8 if args.cache_int8 else binding.KVF_CACHE_INT4 if args.cache_int4 else 0
    cfg = binding.make_config(H, Hkv, d, "bf16", P + nq + ndec, 2048, rope_base=w.rope_base, flags=flags)
    cache = binding.Cache(cfg)
    gen = torch.Generator(device="cuda").manual_seed(args.seed)

    def draw(tokens, heads):
        return torch.randn((tokens, heads, d), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)

    fq, fk, fv = draw(2048, H), draw(2048, Hkv), draw(2048, Hkv)
    fout = torch.empty_like(fq)
    h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    h0.record()
    for _ in range(P // 2048):
        cache.fold_step(fq, fk, fv, out=fout)
    h1.record()
    torch.cuda.synchronize()
    haystack_ms = h0.elapsed_time(h1)
    del fq, fk, fv, fout
    qs = [(draw(nq, H), draw(nq, Hkv), draw(nq, Hkv)) for _ in range(K)]
    dq, dk, dv = draw(1, H), draw(1, Hkv), draw(1, Hkv)
    out_q, out_d = torch.empty((nq, H, d), dtype=torch.bfloat16, device="cuda"), torch.empty((1, H, d), dtype=torch.bfloat16, device="cuda")

    def questions():
        for q, k, v in qs:
            cache.fold_step(q, k, v, out=out_q)
            for _ in range(ndec):
                cache.fold_step(dq, dk, dv, out=out_d)
            cache.set_len(P)

    for _ in range(max(args.warmup, 3)):
        questions()
    torch.cuda.synchronize()
    launches0 = cache.launch_count()
    sampler = ClockSampler(0)
    sampler.start()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    reps = max(args.steps, 1) * 4                                    # a timed stretch of about half a second
    for _ in range(reps):
        questions()
    b.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = a.elapsed_time(b) / reps
    assert cache.status() == binding.KVF_OK, hex(cache.status_word())
    row_bytes = 2 * Hkv * ((d + 4) if args.cache_int8 else (d // 2 + 4) if args.cache_int4 else 2 * d)
    rows = (P + nq) + sum(P + nq + i + 1 for i in range(ndec))       # cache rows the steps of one question read
    gbs = K * rows * row_bytes / (ms * 1e-3) / 1e9
    pk = peaks()
    line = {"metric": "fold-step tokens/s", "value": K * (nq + ndec) / (ms * 1e-3), "unit": "tokens/s", "n_gpus": 1,
            "steps": reps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "multi_needle", "haystack_tokens": P, "questions_per_step": K, "question_tokens": nq,
                       "decoded_tokens": ndec, "n_q_heads": H, "n_kv_heads": Hkv, "head_dim": d,
                       "cache_storage": "int8 codes + fp32 row scales" if args.cache_int8 else
                                        "int4 codes + fp32 row scales" if args.cache_int4 else "bf16 rows",
                       "launch": "one kvf_fold_step per question chunk and per decoded token, kvf_cache_set_len back to "
                                 "the haystack after every question",
                       "l2": "inputs larger than L2 (%.0f MB of cache rows per step)" % (P * row_bytes / 1e6)},
            "ms_per_question": ms / K,
            "haystack_fold_ms": haystack_ms,
            "haystack_fold_note": "the haystack folded once in chunks of 2048, outside the timed region: what every "
                                  "further question would cost again without kvf_cache_set_len",
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": gbs / pk["hbm_gbs"],
                         "peak_source": "measured copy bandwidth" if pk["_source"] == "measured" else "fallback copy bandwidth",
                         "traffic": None, "kernel": "whole steps (rotate + append, attention, merge)",
                         "cache_bytes_per_question": rows * row_bytes},
            "cpu_baseline": None, "e2e": None, "gpu_launches": cache.launch_count() - launches0, "clocks": clocks}
    print(json.dumps(line), flush=True)


def run_row_range(args):
    """One sequence whose cache rows are dealt to the ranks chunk by chunk (not the headline line; strong
    scaling: the whole job is one chain).  Every step: the rank that takes the chunk folds it, the others let the
    same queries attend to the rows they hold (kvf_attend), one all-gather of (out, lse) and kvf_merge_partials
    (multi.row_range_fold_step).  On one GPU the owner is always rank 0 and the gather is the identity: the line
    then shows what the split costs a step (the log-sum-exp output, fp32 parts and the merge kernel)."""
    import torch.distributed as dist
    from paper_2605_12471_b200 import binding, multi
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the fold step has no CPU path")
    rank, world, local = multi.env_rank()
    torch.cuda.set_device(local)
    if world > 1 and not dist.is_initialized():
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    w = workloads.DEEP_CHAIN
    if args.tokens or args.chunk:
        w = w.with_(tokens=args.tokens or w.tokens, chunk=args.chunk or w.chunk)
    T, C, H, Hkv, d = w.tokens, w.chunk, w.n_q_heads, w.n_kv_heads, w.head_dim
    N = T // C
    mine = (N + world - 1 - rank) // world * C + C           # rows this rank will hold, rounded up
    flags = binding.KVF_OUT_F32                               # parts travel in fp32: no second rounding in the merge
    cfg = binding.make_config(H, Hkv, d, "bf16", min(T, mine), C, rope_base=w.rope_base, flags=flags)
    cache = binding.Cache(cfg)
    q, k, v = workloads.sequence_inputs(w, args.seed, sequence=0, device="cuda")      # every rank draws the same sequence

    def chain():
        cache.reset()
        for t in range(N):
            sl = slice(t * C, (t + 1) * C)
            multi.row_range_fold_step(cache, q[sl], k[sl], v[sl], t, t * C, rank, world)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(3):
        chain()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    a.record()
    for _ in range(args.steps):
        chain()
    b.record()
    barrier()
    ms = multi.max_over_ranks(a.elapsed_time(b), device="cuda") / args.steps
    clocks = sampler.stop() if rank == 0 else None
    assert cache.status() == binding.KVF_OK, hex(cache.status_word())
    if rank == 0:
        pk = peaks()
        tf = w.flops_chain() / (ms * 1e-3) / 1e12
        line = {"metric": "fold-step tokens/s", "value": T / (ms * 1e-3), "unit": "tokens/s", "n_gpus": world,
                "steps": args.steps, "warmup": 3, "ms_per_step": ms, "higher_is_better": True, "scaling": "strong",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": "row_range_" + w.name, "shard": "cache rows, chunk t on rank t % world", "tokens": T,
                           "chunk": C, "n_q_heads": H, "n_kv_heads": Hkv, "head_dim": d,
                           "exchange": "all-gather of fp32 (out, lse): %d bytes per rank and step" % (C * H * (d + 1) * 4),
                           "launch": "every step from the host", "l2": "inputs larger than L2 at full size"},
                "attention_tflops": tf,
                "roofline": {"bound": "tensor", "achieved": tf, "peak": pk["bf16_tflops_sustained"] * world,
                             "unit": "TFLOP/s", "frac": tf / (pk["bf16_tflops_sustained"] * world),
                             "peak_source": "measured sustained bf16 x ranks" if pk["_source"] == "measured" else "fallback x ranks",
                             "kernel": "whole chain (all kernels, exchange and merge)", "traffic": None},
                "cpu_baseline": None, "e2e": None, "gpu_launches": cache.launch_count() // (args.steps + 3) + N,
                "clocks": clocks}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--tokens", type=int, default=0, help="shorter chain (debugging; not the benchmark workload)")
    ap.add_argument("--chunk", type=int, default=0)
    ap.add_argument("--prefill", type=int, default=0,
                    help="tokens folded (in 2048-token steps, untimed) before every timed chain: the timed chain "
                         "then runs from this prefix to --tokens (decode- and question-shaped steps at depth)")
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f32"],
                    help="cache and input dtype (not the benchmark workload)")
    ap.add_argument("--workload", default="deep_chain", choices=["deep_chain", "llama_16k", "sweep", "full_stack", "batch_decode", "multi_needle", "row_range"],
                    help="deep_chain: 131 072 tokens in chunks of 256 (the headline line).  llama_16k: 16 384 tokens "
                         "in chunks of 2048, inputs scaled by 1/sqrt(128).  sweep: 65 536 tokens at chunks of 128, "
                         "512, 2048 and 8192, each with a bf16 and an fp32 cache, one line per combination with the "
                         "output drift against the oracle on sampled rows.  full_stack: the 4 x 32-layer "
                         "memory-scale fold (64 GiB of cache; a separate, longer run).  batch_decode: --caches paged "
                         "caches of --prefill tokens each decoding --chunk tokens per batch step (with --cache-int8 / "
                         "--cache-int4 on quantised pages)")
    ap.add_argument("--q-heads", type=int, default=0,
                    help="query heads of the layer (with --kv-heads: another model's attention shape, e.g. 28 / 4 for "
                         "Qwen2.5-7B; not the benchmark workload)")
    ap.add_argument("--kv-heads", type=int, default=0)
    ap.add_argument("--caches", type=int, default=32, help="batch_decode: sequences decoded together")
    ap.add_argument("--needles", type=int, default=8,
                    help="multi_needle: questions asked one after the other about one folded haystack (--prefill tokens), "
                         "each a chunk of --chunk tokens and 30 decoded tokens, with kvf_cache_set_len back in between")
    ap.add_argument("--sequences", type=int, default=4)
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--seed", type=int, default=2605)
    ap.add_argument("--ref-rows", type=int, default=16)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--force-simt", action="store_true")
    ap.add_argument("--paged", action="store_true", help="keep the cache in shuffled 128-token pages of a pool")
    ap.add_argument("--cache-int8", action="store_true",
                    help="store the cache as int8 codes + one fp32 scale per row (KVF_CACHE_INT8); byte counts in the "
                         "output line then count 132 bytes per cached row instead of 256")
    ap.add_argument("--cache-int4", action="store_true", help="the same with 4-bit codes (68 bytes per cached row)")
    ap.add_argument("--shard", default="sequences", choices=["sequences", "kv_heads"],
                    help="with --gpus N: one sequence per rank (weak scaling), or ONE sequence whose KV heads and "
                         "the query heads that read them are dealt to the ranks (strong scaling, no exchange)")
    ap.add_argument("--sinks", type=int, default=0)
    ap.add_argument("--window", type=int, default=0,
                    help="sink + window mask (the paper's StreamingLLM comparison runs 4 + 1020); 0 = full prefix. "
                         "FLOP and byte counts in the output line then count the visible keys only")
    ap.add_argument("--batched", action="store_true",
                    help="full_stack only: the caches live in one paged pool and every chunk is one batch step")
    ap.add_argument("--no-combine-behind", action="store_true",
                    help="leave the merge of a step's partial results on the caller's stream (no KVF_COMBINE_BEHIND)")
    ap.add_argument("--no-graph", action="store_true",
                    help="launch every fold step of the timed chains from the host instead of replaying the chain "
                         "as one CUDA graph captured from the same kvf_fold_step calls")
    return ap.parse_args()


def main():
    args = parse_args()
    if args.workload == "full_stack" and args.impl == "ours":
        run_full_stack(args)
        return
    if args.workload == "batch_decode" and args.impl == "ours":
        run_batch_decode(args)
        return
    if args.workload == "multi_needle" and args.impl == "ours":
        run_multi_needle(args)
        return
    if args.workload == "row_range" and args.impl == "ours":
        run_row_range(args)
        return
    if args.workload == "sweep":
        variants = workloads.SWEEP
    elif args.workload == "llama_16k":
        variants = [workloads.LLAMA_16K]
    else:
        variants = [workloads.DEEP_CHAIN]
    for w in variants:
        if args.tokens or args.chunk or args.prefill or (args.dtype != w.dtype and args.workload != "sweep"):
            w = w.with_(name=f"chain_{args.tokens or w.tokens}_c{args.chunk or w.chunk}_from_{args.prefill}_{args.dtype}",
                        tokens=args.tokens or w.tokens, chunk=args.chunk or w.chunk, dtype=args.dtype)
        if args.q_heads or args.kv_heads:
            w = w.with_(name=f"{w.name}_heads_{args.q_heads or w.n_q_heads}_{args.kv_heads or w.n_kv_heads}",
                        n_q_heads=args.q_heads or w.n_q_heads, n_kv_heads=args.kv_heads or w.n_kv_heads)
        if args.impl == "reference":
            run_reference(args, w)
        else:
            run_chain_bench(args, w, drift=(args.workload == "sweep"))
            torch.cuda.empty_cache()                     # a sweep's next variant starts from an empty pool
    if args.impl == "ours" and int(os.environ.get("WORLD_SIZE", "1")) > 1:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()


def oracle_drift(w, seed, q, k, v, out, C, budget_steps=15, rows_extra=10):
    """Output drift against the fp64 oracle on sampled rows of sampled steps of one chain (the
    oracle ingests every chunk, so it holds the same history as the cache), and the oracle's own
    speed on those rows.  q, k, v, out hold the whole chain on the device."""
    import numpy as np

    import oracle
    N = w.tokens // C
    rng = np.random.default_rng(seed + C)
    steps = {0, 1, 2, N // 4, N // 2, N - 2, N - 1}
    steps = {t for t in steps if 0 <= t < N}
    steps.update(int(x) for x in rng.integers(0, N, size=max(0, budget_steps - len(steps))))
    oc = oracle.OracleCache(w.n_q_heads, w.n_kv_heads, w.head_dim, w.tokens, rope_base=w.rope_base)
    per_step, cpu_s, pairs = [], 0.0, 0
    worst, sum_abs, count = 0.0, 0.0, 0
    for t in range(N):
        sl = slice(t * C, (t + 1) * C)
        qc, kc, vc = (x[sl].to("cpu", torch.float64).numpy() for x in (q, k, v))
        if t not in steps:
            oc.fold_step(qc, kc, vc, rows=[])
            continue
        rows = sorted({r for r in (0, 1, C // 2 - 1, C // 2, C - 2, C - 1) if 0 <= r < C} |
                      {int(x) for x in rng.integers(0, C, size=rows_extra)})
        p0 = len(oc)
        t0 = time.perf_counter()
        ref = oc.fold_step(qc, kc, vc, rows=rows)
        cpu_s += time.perf_counter() - t0
        pairs += sum(p0 + r + 1 for r in rows)
        got = out[sl][rows].to("cpu", torch.float64).numpy()
        err = np.abs(got - ref)
        per_step.append({"step": t, "prefix": t * C, "max_abs": float(err.max()), "mean_abs": float(err.mean()),
                         "rel_rms": float(np.sqrt((err ** 2).sum() / max((ref ** 2).sum(), 1e-300)))})
        worst, sum_abs, count = max(worst, float(err.max())), sum_abs + float(err.sum()), count + err.size
    return {"max_abs": worst, "mean_abs": sum_abs / max(count, 1), "checked_steps": len(per_step),
            "rows_per_step": 6 + rows_extra, "per_step": per_step}, pairs / max(cpu_s, 1e-9), cpu_s


def run_chain_bench(args, w, drift=False):
    from paper_2605_12471_b200 import binding, multi
    import torch.distributed as dist

    rank, world, local = multi.env_rank()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the fold step has no CPU path")
    torch.cuda.set_device(local)
    if world > 1 and not dist.is_initialized():
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    lib = binding.load()
    steps_timed = args.steps if not drift else max(1, min(args.steps, 3))

    T, C = w.tokens, w.chunk
    P0 = args.prefill
    if P0 % 2048 or (T - P0) % C or P0 >= T:
        raise SystemExit("--prefill must be a multiple of 2048 below --tokens, and (tokens - prefill) a multiple of the chunk")
    N = (T - P0) // C                                  # timed fold steps per chain
    by_heads = args.shard == "kv_heads"
    seq = 0 if by_heads else multi.sequence_of_rank(rank)[0]
    wt = w.with_(tokens=T - P0)                        # the timed part's inputs
    q, k, v = workloads.sequence_inputs(wt, args.seed, sequence=seq, device="cuda")
    if by_heads:
        # every rank draws the whole sequence and keeps its heads; from here on `w` is the rank's shape
        q, k, v = multi.shard_heads(q, k, v, rank, world)
        w = w.with_(n_q_heads=q.shape[1], n_kv_heads=k.shape[1])
    H, Hkv, d = w.n_q_heads, w.n_kv_heads, w.head_dim
    out = torch.empty_like(q)
    # (the two host-step flags touch kvf_fold_step_host only: uploads ahead of, result copies behind the steps;
    # KVF_COMBINE_BEHIND puts the merge of a step's partial results beside the next step's rotate + append
    # kernel - a chain ends with kvf_cache_flush, inside the timed region)
    flags = (binding.KVF_FORCE_SIMT if args.force_simt else 0) | binding.KVF_HOST_UPLOAD_AHEAD | binding.KVF_HOST_DOWNLOAD_BEHIND
    if not args.no_combine_behind:
        flags |= binding.KVF_COMBINE_BEHIND
    if args.cache_int8:
        flags |= binding.KVF_CACHE_INT8
    if args.cache_int4:
        flags |= binding.KVF_CACHE_INT4
    if args.paged:
        cfg = binding.make_config(H, Hkv, d, w.dtype, T, max(C, 2048 if P0 else C), rope_base=w.rope_base, flags=flags)
        n_table = (T + 127) // 128
        table = torch.randperm(n_table, generator=torch.Generator().manual_seed(args.seed)).to(torch.int32).cuda()
        pool = torch.empty(binding.paged_pool_bytes(cfg, n_table), dtype=torch.uint8, device="cuda")
        cache = binding.PagedCache(cfg, pool, n_table, table)
    else:
        cache = binding.cache_for(w, flags=flags, max_chunk=max(C, 2048 if P0 else C))
    if args.window:
        cache.set_window(args.sinks, args.window)
    h = cache._h
    launch_stream = [torch.cuda.current_stream().cuda_stream]
    eb = q.element_size()
    qs, ks = C * H * d * eb, C * Hkv * d * eb
    qp, kp, vp, op = q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr()
    if P0:
        fq, fk, fv = workloads.chunk_inputs(w.with_(chunk=2048), args.seed + 1, 0, sequence=seq + rank, device="cuda")
        fout = [torch.empty_like(fq), torch.empty_like(fq)]       # (a step's results stay the library's until the next step ends)

    # bytes a step reads per cached token: K and V rows of every KV head (int8: d codes + one fp32 scale per row)
    bytes_per_token = (2 * Hkv * (d + 4) if args.cache_int8 else 2 * Hkv * (d // 2 + 4) if args.cache_int4
                       else w.cache_bytes_per_token())

    def visible(prefix):
        """Rows before a chunk that its queries see (all of them without a window)."""
        if args.window and prefix - args.window > args.sinks:
            return args.sinks + args.window
        return prefix

    def prefill():
        """Empty accumulator, then (outside every timed region) the prefix in 2048-token steps."""
        cache.reset()
        for t in range(P0 // 2048):
            cache.fold_step(fq, fk, fv, out=fout[t & 1])
        cache.flush()

    def body(first=0, last=None):
        for t in range(first, N if last is None else last):
            rc = lib.kvf_fold_step(h, qp + t * qs, kp + t * ks, vp + t * ks, C, P0 + t * C, op + t * qs, None,
                                   launch_stream[0])
            if rc:
                raise binding.KvfError(rc, "kvf_fold_step")
        rc = lib.kvf_cache_flush(h, launch_stream[0])      # the last step's merge, if it runs on the library's stream
        if rc:
            raise binding.KvfError(rc, "kvf_cache_flush")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        """K chains between one pair of barriers; with a prefill, one bracket per chain so that the
        prefill stays outside."""
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if P0 == 0:
            barrier()
            a.record()
            for _ in range(steps):
                cache.reset()
                fn()
            b.record()
            barrier()
            return multi.max_over_ranks(a.elapsed_time(b), device="cuda")
        total = 0.0
        for _ in range(steps):
            prefill()
            barrier()
            a.record()
            fn()
            b.record()
            barrier()
            total += a.elapsed_time(b)
        return multi.max_over_ranks(total, device="cuda")

    for _ in range(args.warmup):
        prefill()
        body()
    # The chain's launches are fixed once the sizes are (every step's prefix is a kernel argument), so the
    # timed chains replay one CUDA graph captured from the very kvf_fold_step calls of body().  The host's
    # row count advances during the capture only; a replay needs no reset.
    graph, run_chain = None, body
    if not args.no_graph:
        prefill()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            launch_stream[0] = torch.cuda.current_stream().cuda_stream
            body()
        launch_stream[0] = torch.cuda.current_stream().cuda_stream
        run_chain = graph.replay
        prefill()
        run_chain()                                      # one untimed replay (uploads the graph)
        torch.cuda.synchronize()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    cyc_a, ns_a = cache.sm_clock()
    ms = timed(run_chain, steps_timed)
    cyc_b, ns_b = cache.sm_clock()
    clocks = sampler.stop() if rank == 0 else None
    assert graph is not None or len(cache) == T
    if cache.status() != binding.KVF_OK:
        raise SystemExit("device status word reports a timed-out wait")
    value = multi.whole_job_tokens_per_s(T - P0, steps_timed, 1 if by_heads else world, ms)

    # per-kernel time of the same chain, CUDA events around every launch on the launching stream;
    # read out in bins of steps, which gives the latency against the prefix length.  The SM clock is
    # read through NVML meanwhile, so every bin carries the clock it ran at: time x clock separates a
    # kernel that got slower from a clock that the power cap lowered.
    prefill()
    torch.cuda.synchronize()
    l0 = cache.launch_count()
    cache.profile(True)
    kms, kcnt, curve = [0.0, 0.0, 0.0], [0, 0, 0], []
    nbins = min(16, N)
    nvml = NvmlClock(local)
    nvml.start()
    t_prof0 = time.perf_counter()
    tensor_shaped = cache.plan(C, T - C)[0] == 1
    per_clock_rate = TENSOR_FLOP_PER_SM_CLOCK / (3.0 if w.dtype == "f32" else 1.0)
    clock_cycles, clock_ns = 0, 0
    for bi in range(nbins):
        first, last = bi * N // nbins, (bi + 1) * N // nbins
        t0 = time.perf_counter()
        cy0, ns0 = cache.sm_clock()
        body(first, last)
        bms, bcnt = cache.profile_read()
        cy1, ns1 = cache.sm_clock()
        t1 = time.perf_counter()
        fl = sum(w.flops_step(visible(P0 + t * C), C) for t in range(first, last))
        by = sum(visible(P0 + t * C) + C for t in range(first, last)) * bytes_per_token
        # the clock the attention kernels of this bin ran at, from the kernels' own cycle and nanosecond counters
        # (the NVML reading is kept beside it: it lags a power-capped clock)
        mhz_nvml = nvml.median_between(t0, t1)
        mhz = 1e3 * (cy1 - cy0) / (ns1 - ns0) if ns1 > ns0 else mhz_nvml
        clock_cycles += cy1 - cy0
        clock_ns += ns1 - ns0
        point = {"prefix_from": P0 + first * C, "prefix_to": P0 + (last - 1) * C,
                 "step_us": 1e3 * sum(bms) / (last - first), "attention_us": 1e3 * bms[1] / (last - first),
                 "attention_tflops": fl / (bms[1] * 1e-3) / 1e12, "cache_read_gbs": by / (bms[1] * 1e-3) / 1e9,
                 "sm_mhz": mhz, "sm_mhz_nvml": mhz_nvml}
        if mhz:
            point["attention_kilocycles"] = 1e3 * bms[1] / (last - first) * mhz / 1e3
            if tensor_shaped:
                point["tensor_flop_per_sm_clock_frac"] = fl / (bms[1] * 1e-3 * mhz * 1e6 * N_SMS * per_clock_rate)
        curve.append(point)
        kms = [x + y for x, y in zip(kms, bms)]
        kcnt = [x + y for x, y in zip(kcnt, bcnt)]
    nvml.stop()
    prof_mhz = 1e3 * clock_cycles / clock_ns if clock_ns else nvml.median_between(t_prof0, time.perf_counter())
    cache.profile(False)
    launches = (cache.launch_count() - l0) * steps_timed       # kernels of the timed chains
    pk = peaks()
    attn_flops = sum(w.flops_step(visible(P0 + t * C), C) for t in range(N))
    attn_tflops = attn_flops / (kms[1] * 1e-3) / 1e12
    cache_bytes_read = sum(visible(P0 + t * C) + C for t in range(N)) * bytes_per_token
    hbm_gbs = cache_bytes_read / (kms[1] * 1e-3) / 1e9
    traffic = None
    if NCU_TRAFFIC_BYTES_PER_CACHE_BYTE is not None and w.dtype == "bf16" and not (args.cache_int8 or args.cache_int4 or args.force_simt):
        traffic = NCU_TRAFFIC_BYTES_PER_CACHE_BYTE * cache_bytes_read / kcnt[1]
    # which roof binds: arithmetic intensity G*C FLOP per cache byte against the ridge of the measured peaks
    ridge = pk["bf16_tflops_sustained"] * 1e12 / (pk["hbm_gbs"] * 1e9)
    intensity = attn_flops / cache_bytes_read
    plan_last = cache.plan(C, T - C)
    if w.dtype == "f32" and not plan_last[0]:
        # CUDA-core kernel (head_dim 64, or forced): the roof is the FFMA rate, 148 SMs x 128 lanes x 2 FLOP at
        # the 1965 MHz maximum clock
        alu_peak = N_SMS * 128 * 2 * 1.965e9 / 1e12
        roofline = {"bound": "alu", "achieved": attn_tflops, "peak": alu_peak, "unit": "TFLOP/s",
                    "frac": attn_tflops / alu_peak, "peak_source": "derived: 148 SMs x 128 FFMA lanes x 2 x 1.965 GHz"}
    elif w.dtype == "f32":
        # fp32 caches on the tensor pipe: every product is three fp16 MMAs (hi x hi, hi x lo, lo x hi of operands
        # split into two fp16 halves), so the roof is a third of the fp16/bf16 rate
        peak = pk["bf16_tflops_sustained"] / 3.0
        roofline = {"bound": "tensor", "achieved": attn_tflops, "peak": peak, "unit": "TFLOP/s", "frac": attn_tflops / peak,
                    "peak_source": pk["_source"] + " sustained bf16 / 3 (three fp16 products per fp32 product)",
                    "gate": "sustained", "frac_sustained": attn_tflops / peak,
                    "frac_burst": attn_tflops / (pk["bf16_tflops"] / 3.0), "frac_nominal": attn_tflops / (NOMINAL["bf16_tflops"] / 3.0)}
    elif intensity >= ridge:
        roofline = {"bound": "tensor", "achieved": attn_tflops, "peak": pk["bf16_tflops_sustained"], "unit": "TFLOP/s",
                    "frac": attn_tflops / pk["bf16_tflops_sustained"], "peak_source": pk["_source"] + " sustained bf16",
                    # the three denominators side by side; the 60 % target is judged on the measured sustained one
                    # (the part is power-capped: a seconds-long bf16 GEMM loop settles there)
                    "gate": "sustained", "frac_sustained": attn_tflops / pk["bf16_tflops_sustained"],
                    "frac_burst": attn_tflops / pk["bf16_tflops"], "frac_nominal": attn_tflops / NOMINAL["bf16_tflops"],
                    "peaks_tflops": {"nominal": NOMINAL["bf16_tflops"], "burst": pk["bf16_tflops"],
                                     "sustained": pk["bf16_tflops_sustained"]}}
    else:
        roofline = {"bound": "hbm", "achieved": hbm_gbs, "peak": pk["hbm_gbs"], "unit": "GB/s",
                    "frac": hbm_gbs / pk["hbm_gbs"], "peak_source": pk["_source"] + " copy bandwidth",
                    "gate": "measured copy", "frac_sustained": hbm_gbs / pk["hbm_gbs"], "frac_burst": hbm_gbs / pk["hbm_gbs"],
                    "frac_nominal": hbm_gbs / NOMINAL["hbm_gbs"]}
    if prof_mhz and roofline["bound"] == "tensor":
        # clock-normalised: share of the tensor pipe's per-clock rate at the clock sampled during this pass
        per_clock = TENSOR_FLOP_PER_SM_CLOCK / (3.0 if w.dtype == "f32" else 1.0)
        roofline["sm_mhz_during_profile"] = prof_mhz
        roofline["frac_of_tensor_rate_at_sampled_clock"] = attn_tflops * 1e12 / (prof_mhz * 1e6 * N_SMS * per_clock)
    if ns_b > ns_a and roofline["bound"] == "tensor":
        # (only the tcgen05 kernels for long chunks keep these counters: not reported for decode-shaped runs)
        # the attention kernels inside the timed chains themselves (no events between the kernels there): time and
        # cycles one CTA of every launch (its last row block) was running, from the kernels' own counters
        in_ms = (ns_b - ns_a) * 1e-6 / steps_timed
        roofline["in_timed_chains"] = {"attention_ms_per_chain": in_ms, "sm_mhz": 1e3 * (cyc_b - cyc_a) / (ns_b - ns_a),
                                       "attention_tflops": attn_flops / (in_ms * 1e-3) / 1e12,
                                       "other_ms_per_chain": ms / steps_timed - in_ms}
    roofline.update({
        "kernel": "prefix+chunk attention", "traffic": traffic, "traffic_source": NCU_TRAFFIC_SOURCE if traffic else None,
        "flops_per_launch": attn_flops / kcnt[1],
        "cache_bytes_per_launch": cache_bytes_read / kcnt[1], "ms_per_launch": kms[1] / kcnt[1], "launches": kcnt[1],
        "kernel_ms_per_chain": {"rope_append": kms[0], "attention": kms[1], "combine": kms[2]},
        "attention_tflops": attn_tflops, "cache_read_gbs": hbm_gbs, "flop_per_cache_byte": intensity,
        "ridge_flop_per_byte": ridge, "hbm_peak_gbs": pk["hbm_gbs"], "bf16_peak_tflops": pk["bf16_tflops_sustained"],
    })

    drift_report = None
    cpu = None
    if drift and rank == 0:
        # one more eager chain whose outputs stay in `out`; the oracle follows it on sampled rows
        cache.reset()
        body()
        torch.cuda.synchronize()
        drift_report, pairs_per_s, cpu_s = oracle_drift(w, args.seed, q, k, v, out, C)
        threads = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
        cpu = {"value": tokens_per_s_from_pairs(w, pairs_per_s, P0), "unit": "tokens/s", "cores": threads, "kind": "oracle",
               "sample": (f"{drift_report['rows_per_step']} query rows x {H} heads at {drift_report['checked_steps']} steps "
                          f"spread over the chain ({cpu_s:.1f} s of CPU work), fp64 oracle; tokens/s extrapolated "
                          f"linearly in visible (query,key) pairs over the chain")}

    e2e = None
    if not args.no_e2e:
        qh, kh, vh = (x.cpu().pin_memory() for x in (q, k, v))
        oh = torch.empty(out.shape, dtype=out.dtype).pin_memory()
        qhp, khp, vhp, ohp = qh.data_ptr(), kh.data_ptr(), vh.data_ptr(), oh.data_ptr()

        def body_host():
            for t in range(N):
                rc = lib.kvf_fold_step_host(h, qhp + t * qs, khp + t * ks, vhp + t * ks, C, P0 + t * C, ohp + t * qs,
                                            None, launch_stream[0])
                if rc:
                    raise binding.KvfError(rc, "kvf_fold_step_host")
            cache.flush()                                    # the chain ends when its last results are in host memory

        prefill()
        body_host()
        e2e_steps = steps_timed                              # as many chains as the device-resident leg
        ems = timed(body_host, e2e_steps)
        e2e = {"value": (1 if by_heads else world) * e2e_steps * (T - P0) / (ems * 1e-3), "unit": "tokens/s", "steps": e2e_steps,
               "h2d_bytes_per_step": (T - P0) * (H + 2 * Hkv) * d * eb, "d2h_bytes_per_step": (T - P0) * H * d * eb,
               "ms_per_step": ems / e2e_steps}

    if cpu is None and rank == 0 and world == 1 and not args.no_cpu_baseline and not args.window:
        rate, times, threads, rows = oracle_rate(w, args.seed, rows_per_step=32, repeats=4, prefix=max(0, T - 5 * C))
        cpu = {"value": tokens_per_s_from_pairs(w, rate, P0), "unit": "tokens/s", "cores": threads, "kind": "oracle",
               "sample": (f"{len(rows)} query rows x {H} heads of one chunk at prefix ~{T - 4 * C}, median of "
                          f"{len(times)} repeats ({sum(times):.1f} s of CPU work), fp64 oracle; tokens/s "
                          f"extrapolated linearly in visible (query,key) pairs over the chain")}
        if set_oracle_threads(1):
            # the same oracle on one thread, on a sample an eighth the size
            rate1, times1, _, rows1 = oracle_rate(w, args.seed, rows_per_step=4, repeats=1, prefix=max(0, T - 5 * C))
            set_oracle_threads(threads)
            cpu["single_thread"] = {"value": tokens_per_s_from_pairs(w, rate1, P0), "unit": "tokens/s", "cores": 1,
                                    "sample": f"{len(rows1)} query rows x {H} heads, one repeat ({sum(times1):.1f} s of CPU work)"}

    if rank == 0:
        step_flops = attn_flops * world * steps_timed
        line = {
            "metric": "fold-step tokens/s", "value": value, "unit": "tokens/s", "n_gpus": world,
            "steps": steps_timed, "warmup": args.warmup, "ms_per_step": ms / steps_timed,
            "higher_is_better": True, "scaling": "strong" if by_heads else "weak", "vs_baseline": None, "dtype": w.dtype,
            "data": "synthetic",
            "config": {"workload": w.name, "shard": args.shard, "tokens": T, "chunk": C, "prefill": P0, "fold_steps_per_step": N,
                       "n_q_heads": H, "n_kv_heads": Hkv, "head_dim": d, "rope_base": w.rope_base,
                       "sequences_per_gpu": 1, "paged": bool(args.paged), "sinks": args.sinks, "window": args.window,
                       "cache_storage": ("int8 codes + fp32 row scales" if args.cache_int8 else
                                         "int4 codes + fp32 row scales" if args.cache_int4 else w.dtype),
                       "launch": "per-step host launches" if graph is None else "one CUDA graph per chain, captured from the same calls",
                       "combine": "on the caller's stream" if args.no_combine_behind else "behind the attention kernel on the library's stream (KVF_COMBINE_BEHIND), chain closed by kvf_cache_flush",
                       "l2": f"inputs larger than L2 (cache grows to {T * bytes_per_token / 2 ** 20:.0f} MiB per chain)",
                       "last_step_plan": {"tensor_core": plan_last[0], "splits": plan_last[1], "ctas": plan_last[2]}},
            "attention_tflops": step_flops / (ms * 1e-3) / 1e12,
            "roofline": roofline, "latency_vs_prefix": curve, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clocks,
        }
        if drift_report is not None:
            line["drift_vs_oracle"] = drift_report
        print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()

"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds no arithmetic of the fold step: it only names the workload
shapes and draws i.i.d. Gaussian Q/K/V from recorded seeds.  Both the CUDA
path's callers and the oracle's callers take their inputs from here, so the two
sides see the same bits.

The paper measures on PG-19 text pushed through trained models (Section 2,
"Three reference conditions"; Section 5, scaling table).  Neither exists here,
so Gaussian tensors with the Llama-3.1-8B attention-layer shape (32 query
heads, 8 KV heads, head_dim 128, chunk 256, up to 131 072 tokens, chain depth
511) stand in for them.
"""
from __future__ import annotations

import dataclasses
import hashlib
from typing import Tuple

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str            # "bf16" or "f32": dtype of q, k, v, the cache and out
    chunk: int            # C
    tokens: int           # T per sequence
    rope_base: float
    input_scale: float = 1.0
    n_sequences: int = 1
    n_layers: int = 1

    @property
    def n_steps(self) -> int:
        return self.tokens // self.chunk

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    def with_(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)

    def flops_step(self, prefix: int, n: int | None = None) -> float:
        """Multiply-adds x2 over visible (query, key) pairs, QK^T and PV."""
        n = self.chunk if n is None else n
        return 4.0 * self.n_q_heads * self.head_dim * (n * prefix + n * (n + 1) / 2)

    def flops_chain(self) -> float:
        t = self.tokens
        return 4.0 * self.n_q_heads * self.head_dim * t * (t + 1) / 2

    def cache_bytes_per_token(self) -> int:
        return 2 * self.n_kv_heads * self.head_dim * (2 if self.dtype == "bf16" else 4)


_LLAMA = dict(n_q_heads=32, n_kv_heads=8, head_dim=128, rope_base=500000.0)

TINY = Workload("tiny_fold", 4, 1, 64, "f32", 64, 512, 10000.0)
LLAMA_16K = Workload("llama8b_16k_c2048", dtype="bf16", chunk=2048, tokens=16384,
                     input_scale=128 ** -0.5, **_LLAMA)
DEEP_CHAIN = Workload("deep_chain_128k_c256", dtype="bf16", chunk=256, tokens=131072, **_LLAMA)
FULL_STACK = Workload("full_stack_4x32_128k_c1024", dtype="bf16", chunk=1024, tokens=131072,
                      n_sequences=4, n_layers=32, **_LLAMA)


def sweep(chunk: int, dtype: str) -> Workload:
    """Chunk-size and precision sweep at 65 536 tokens."""
    return Workload(f"sweep_64k_c{chunk}_{dtype}", dtype=dtype, chunk=chunk, tokens=65536, **_LLAMA)


SWEEP = [sweep(c, dt) for c in (128, 512, 2048, 8192) for dt in ("bf16", "f32")]

CONFIGS = [TINY, LLAMA_16K, DEEP_CHAIN, SWEEP, FULL_STACK]


def seed_for(base_seed: int, workload: str, sequence: int, layer: int, step: int) -> int:
    """A 63-bit seed from (base seed, workload name, sequence, layer, step)."""
    h = hashlib.sha256(f"{base_seed}|{workload}|{sequence}|{layer}|{step}".encode()).digest()
    return int.from_bytes(h[:8], "little") & ((1 << 63) - 1)


def chunk_inputs(w: Workload, base_seed: int, step: int, sequence: int = 0, layer: int = 0,
                 device: str | torch.device = "cpu", n_tokens: int | None = None
                 ) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """q [n,H,d], k [n,Hkv,d], v [n,Hkv,d] of one chunk, in the workload's dtype.

    Values are N(0,1) * input_scale drawn in fp32 and rounded once to the dtype.
    The stream depends on the device kind (CPU and CUDA generators differ), so a
    comparison draws on one device and copies to the other.
    """
    n = w.chunk if n_tokens is None else n_tokens
    gen = torch.Generator(device=device)
    gen.manual_seed(seed_for(base_seed, w.name, sequence, layer, step))
    out = []
    for heads in (w.n_q_heads, w.n_kv_heads, w.n_kv_heads):
        x = torch.randn((n, heads, w.head_dim), generator=gen, device=device, dtype=torch.float32)
        if w.input_scale != 1.0:
            x = x * w.input_scale
        out.append(x.to(w.torch_dtype).contiguous())
    return out[0], out[1], out[2]


def sequence_inputs(w: Workload, base_seed: int, sequence: int = 0, layer: int = 0,
                    device: str | torch.device = "cpu"
                    ) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """The whole sequence, as the concatenation of its chunks' inputs."""
    parts = [chunk_inputs(w, base_seed, t, sequence, layer, device) for t in range(w.n_steps)]
    return tuple(torch.cat([p[i] for p in parts], dim=0) for i in range(3))

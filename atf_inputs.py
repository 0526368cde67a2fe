"""Seeded synthetic inputs for the windowed-attention tests and benchmarks.

This module only draws random numbers and names workload shapes.  It holds none of the
method's arithmetic (no RoPE, no window rule, no attention): both the CPU oracle's tests and
the CUDA path's tests/bench take their tensors from here so that they see the same data.

Workloads mirror the attention-layer shapes the paper evaluates (Qwen2.5-0.5B,
Llama-3.2-3B, Qwen2.5-7B-1M); the paper's documents are replaced by i.i.d. N(0,1) values
rounded to bf16, which is legitimate because the method's cost does not depend on the data.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch

SEED0 = 2608029470

LLAMA3_SCALING = {"kind": "llama3", "factor": 32.0, "low_freq_factor": 1.0,
                  "high_freq_factor": 4.0, "original_ctx": 8192}


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    Hq: int
    Hkv: int
    d: int
    N: int            # prefill length, or KV-cache length L for decode
    base: float
    k: float = 2.0
    scaling: dict | None = field(default=None, hash=False, compare=False)
    seed: int = SEED0
    outlier: bool = False   # scale the 4 lowest-frequency pairs of Q and K by 8 (before RoPE)


def tiny(N=2048, k=2.0):
    return Workload("tiny", 1, 2, 1, 64, N, 1e6, k, None, SEED0 + 1)


def qwen05b(N, outlier=False):
    return Workload("qwen2.5-0.5b", 1, 14, 2, 64, N, 1e6, 2.0, None, SEED0 + (3 if outlier else 2), outlier)


def llama32_3b(N, B=1, seed_off=4, outlier=False):
    return Workload("llama-3.2-3b", B, 24, 8, 128, N, 5e5, 2.0, LLAMA3_SCALING, SEED0 + seed_off, outlier)


def qwen7b_1m(N):
    return Workload("qwen2.5-7b-1m", 1, 28, 4, 128, N, 1e7, 2.0, None, SEED0 + 11)


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def normal_bf16(shape, seed, device="cpu"):
    """i.i.d. N(0,1) drawn in fp32 with the given seed, rounded to bf16 (round to nearest even)."""
    g = _gen(device, seed)
    return torch.randn(shape, generator=g, dtype=torch.float32, device=device).to(torch.bfloat16)


def normal_f32(shape, seed, device="cpu"):
    """i.i.d. N(0,1) in fp32 with the given seed (the same draws normal_bf16 rounds)."""
    g = _gen(device, seed)
    return torch.randn(shape, generator=g, dtype=torch.float32, device=device)


def prefill_inputs_f32(w: Workload, device="cpu"):
    """Un-rotated Q, K in fp32 and V in bf16 for the split-precision prefill (same seeds as prefill_inputs)."""
    Q = normal_f32((w.B, w.Hq, w.N, w.d), w.seed * 3 + 0, device)
    K = normal_f32((w.B, w.Hkv, w.N, w.d), w.seed * 3 + 1, device)
    V = normal_bf16((w.B, w.Hkv, w.N, w.d), w.seed * 3 + 2, device)
    if w.outlier:
        h = w.d // 2
        for t in (Q, K):
            t[..., h - 4:h] *= 8
            t[..., w.d - 4:w.d] *= 8
    return Q, K, V


def prefill_inputs(w: Workload, device="cpu"):
    """Un-rotated Q [B,Hq,N,d], K, V [B,Hkv,N,d] in bf16.  RoPE is applied by the caller."""
    Q = normal_bf16((w.B, w.Hq, w.N, w.d), w.seed * 3 + 0, device)
    K = normal_bf16((w.B, w.Hkv, w.N, w.d), w.seed * 3 + 1, device)
    V = normal_bf16((w.B, w.Hkv, w.N, w.d), w.seed * 3 + 2, device)
    if w.outlier:
        h = w.d // 2
        for t in (Q, K):
            t[..., h - 4:h] *= 8     # exact in bf16 (power of two)
            t[..., w.d - 4:w.d] *= 8
    return Q, K, V


def decode_inputs(w: Workload, device="cpu"):
    """q [B,Hq,d], post-RoPE Kcache and Vcache [B,Hkv,L,d], all bf16 N(0,1) drawn directly."""
    q = normal_bf16((w.B, w.Hq, w.d), w.seed * 3 + 0, device)
    Kc = normal_bf16((w.B, w.Hkv, w.N, w.d), w.seed * 3 + 1, device)
    Vc = normal_bf16((w.B, w.Hkv, w.N, w.d), w.seed * 3 + 2, device)
    return q, Kc, Vc


def to_f64(t: torch.Tensor):
    """Exact widening of a bf16 tensor to a float64 NumPy array (host)."""
    return t.detach().to("cpu", torch.float32).numpy().astype("float64")


def sample_rows(N, W, n_random, seed, tile=128):
    """Query rows worth checking at size N: first and last tile, rows next to every window
    boundary that falls inside the sequence, and n_random seeded random rows."""
    rows = set(range(min(tile, N))) | set(range(max(0, N - tile), N))
    for w in W:
        w = int(w)
        for r in (w - 1, w, w + 1, w + 2):
            if 0 <= r < N:
                rows.add(r)
    g = _gen("cpu", seed)
    rows |= set(torch.randint(0, N, (n_random,), generator=g).tolist())
    return sorted(rows)

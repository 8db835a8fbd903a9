"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU oracle.

This module holds shapes, seeds and random draws only -- none of the method's arithmetic
(no mask, no softmax, no layout).  Tensors are drawn on the CPU with a seeded torch generator
as fp32 N(0,1), optionally scaled, and rounded to bf16 (round-to-nearest-even); both the oracle
and the CUDA path read exactly these bf16 values.

The shapes follow the paper's efficiency workload (a 7B-class GQA model: 28 query heads,
4 KV heads, head_dim 128, contexts of 16K-128K tokens, Section 4.5); the paper's datasets and
weights are not needed for the attention operator, so i.i.d. Gaussian tensors stand in.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Tuple

import numpy as np
import torch


@dataclass(frozen=True)
class PrefillWorkload:
    name: str
    batch: int
    seq_len: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    block: int
    window_blocks: int
    sink_blocks: int
    seed: int
    k_scale: float = 1.0  # multiplies K before bf16 rounding (sets the logit spread)

    @property
    def softmax_scale(self) -> float:
        return 1.0 / float(np.sqrt(self.head_dim))


@dataclass(frozen=True)
class DecodeWorkload:
    name: str
    batch: int
    max_len: int
    min_len: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    block: int
    window_blocks: int
    sink_blocks: int
    seed: int
    lens_seed: int

    @property
    def softmax_scale(self) -> float:
        return 1.0 / float(np.sqrt(self.head_dim))


# The paper's default pattern: 5-block local window, 1 block of initial tokens (Section 4.1).
PAPER_WINDOW_BLOCKS = 5
PAPER_SINK_BLOCKS = 1

TINY_PREFILL = PrefillWorkload("tiny_prefill_2k", 1, 2048, 2, 2, 64, 64, 1, 1, seed=1001)
PREFILL_32K = PrefillWorkload("prefill_32k_gqa28x4_d128", 1, 32768, 28, 4, 128, 64,
                              PAPER_WINDOW_BLOCKS, PAPER_SINK_BLOCKS, seed=2002, k_scale=3.0)
PREFILL_128K = PrefillWorkload("prefill_128k_gqa28x4_d128", 1, 131072, 28, 4, 128, 64,
                               PAPER_WINDOW_BLOCKS, PAPER_SINK_BLOCKS, seed=3003)
DECODE_B8 = DecodeWorkload("decode_b8_64k_128k_gqa28x4_d128", 8, 131072, 65536, 28, 4, 128, 64,
                           PAPER_WINDOW_BLOCKS, PAPER_SINK_BLOCKS, seed=4004, lens_seed=4005)

SWEEP_SEQ_LENS = (4096, 8192, 16384, 32768, 65536, 131072, 262144)


def sweep_workload(seq_len: int) -> PrefillWorkload:
    return PrefillWorkload(f"sweep_{seq_len // 1024}k_gqa28x4_d128", 1, seq_len, 28, 4, 128, 64,
                           PAPER_WINDOW_BLOCKS, PAPER_SINK_BLOCKS,
                           seed=5000 + int(np.log2(seq_len)))


def bf16_randn(shape: Tuple[int, ...], seed: int, scale: float = 1.0,
               pin: bool = False) -> torch.Tensor:
    """fp32 N(0,1) * scale from a seeded CPU generator, rounded to bf16."""
    g = torch.Generator(device="cpu").manual_seed(int(seed))
    out = torch.empty(shape, dtype=torch.bfloat16, pin_memory=pin)
    flat = out.view(-1)
    n = flat.numel()
    chunk = 1 << 24  # bounded fp32 staging
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        x = torch.randn(e - s, generator=g, dtype=torch.float32)
        if scale != 1.0:
            x.mul_(scale)
        flat[s:e] = x.to(torch.bfloat16)
    return out


def prefill_inputs(w: PrefillWorkload, pin: bool = False):
    """Q [batch, N, Hq, D], K, V [batch, N, Hkv, D] bf16 on the CPU."""
    q = bf16_randn((w.batch, w.seq_len, w.n_q_heads, w.head_dim), w.seed, pin=pin)
    k = bf16_randn((w.batch, w.seq_len, w.n_kv_heads, w.head_dim), w.seed + 1, w.k_scale, pin=pin)
    v = bf16_randn((w.batch, w.seq_len, w.n_kv_heads, w.head_dim), w.seed + 2, pin=pin)
    return q, k, v


def decode_lens(w: DecodeWorkload) -> np.ndarray:
    """Per-sequence cache lengths, uniform integers in [min_len, max_len], current token included."""
    rng = np.random.Generator(np.random.PCG64(w.lens_seed))
    return rng.integers(w.min_len, w.max_len + 1, size=w.batch, dtype=np.int64)


def decode_inputs(w: DecodeWorkload, pin: bool = False):
    """q [batch, Hq, D], K/V caches [batch, max_len, Hkv, D] bf16 on the CPU, lens [batch]."""
    q = bf16_randn((w.batch, w.n_q_heads, w.head_dim), w.seed, pin=pin)
    kc = bf16_randn((w.batch, w.max_len, w.n_kv_heads, w.head_dim), w.seed + 1, pin=pin)
    vc = bf16_randn((w.batch, w.max_len, w.n_kv_heads, w.head_dim), w.seed + 2, pin=pin)
    return q, kc, vc, decode_lens(w)

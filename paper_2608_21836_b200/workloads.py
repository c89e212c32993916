"""Seeded synthetic workloads shaped like LLM prefill and decode.

This module holds NONE of the method's arithmetic: it only draws bf16 tensors with
PyTorch's CPU generator and names the five benchmark configurations. Both the CUDA
path and the test oracle are fed from here, so that they see identical inputs.

The paper's own workloads (real prompts through Llama-2 / Qwen3 checkpoints) are not
available; these inputs take the head geometry of those model families (GQA 32/8/128,
a small MHA 12/12/64) and stand in for them.

Recipe (every config): ``torch.Generator().manual_seed(seed)``; ``torch.randn`` in
fp32 in the order q, k, v (or q, cache_k, cache_v); multiply by ``value_scale``;
round to bf16. "Prefill then decode" configs draw the whole sequence of S+T tokens at
once: prefill consumes tokens [0, S), decode step t consumes token S+t.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Optional

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    Hq: int
    Hkv: int
    D: int
    value_scale: float = 1.0
    # prefill part (0 = none)
    prefill_B: int = 0
    prefill_S: int = 0
    decode_steps: int = 0          # T: decode steps that follow the prefill
    # stand-alone decode part (0 = none)
    decode_B: int = 0
    decode_len_lo: int = 0         # kv_len drawn uniformly in [lo, hi], both inclusive
    decode_len_hi: int = 0
    decode_Lmax: int = 0
    description: str = ""

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.D)

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv


WORKLOADS = {
    w.name: w
    for w in [
        Workload("tiny", 1001, Hq=4, Hkv=2, D=64, prefill_B=1, prefill_S=128, decode_steps=16,
                 description="B=1 causal prefill of 128 tokens then 16 decode steps"),
        Workload("layer8b", 1002, Hq=32, Hkv=8, D=128, value_scale=0.5, prefill_B=1,
                 prefill_S=2048, decode_steps=256,
                 description="8B-shaped layer: prefill 2048 then 256 decode steps, contiguous cache"),
        Workload("batched_decode", 1003, Hq=32, Hkv=8, D=128, decode_B=32, decode_len_lo=512,
                 decode_len_hi=4096, decode_Lmax=4096,
                 description="B=32 ragged decode, kv_len uniform in [512, 4096]"),
        Workload("long_prefill", 1004, Hq=32, Hkv=8, D=128, prefill_B=4, prefill_S=8192,
                 description="B=4 causal prefill of 8192 tokens with the cache written in the same pass"),
        Workload("mha_small", 1005, Hq=12, Hkv=12, D=64, prefill_B=8, prefill_S=512,
                 decode_B=64, decode_len_lo=1024, decode_len_hi=1024, decode_Lmax=1024,
                 description="MHA small model: prefill B=8 S=512, decode B=64 at context 1024"),
    ]
}


def _randn_bf16(shape, gen: torch.Generator, value_scale: float) -> torch.Tensor:
    x = torch.randn(shape, generator=gen, dtype=torch.float32)
    if value_scale != 1.0:
        x.mul_(value_scale)
    return x.to(torch.bfloat16)


#: bf16 quiet-NaN bit pattern used to poison memory that must never reach the math
NAN_BITS = 0x7FC0


def nan_like(shape) -> torch.Tensor:
    return torch.full(shape, NAN_BITS, dtype=torch.int16).view(torch.bfloat16)


@dataclass
class Sequence:
    """q [B, S+T, Hq, D], k and v [B, S+T, Hkv, D] for a prefill followed by T decode steps."""
    w: Workload
    q: torch.Tensor
    k: torch.Tensor
    v: torch.Tensor
    S: int
    T: int


def make_sequence(w: Workload, S: Optional[int] = None, T: Optional[int] = None,
                  B: Optional[int] = None, seed: Optional[int] = None) -> Sequence:
    S = w.prefill_S if S is None else S
    T = w.decode_steps if T is None else T
    B = w.prefill_B if B is None else B
    gen = torch.Generator().manual_seed(w.seed if seed is None else seed)
    q = _randn_bf16((B, S + T, w.Hq, w.D), gen, w.value_scale)
    k = _randn_bf16((B, S + T, w.Hkv, w.D), gen, w.value_scale)
    v = _randn_bf16((B, S + T, w.Hkv, w.D), gen, w.value_scale)
    return Sequence(w, q, k, v, S, T)


@dataclass
class DecodeBatch:
    """q [B, Hq, D]; caches [B, Hkv, Lmax, D] whose slots >= kv_len[b] hold NaN; kv_len [B] int32."""
    w: Workload
    q: torch.Tensor
    cache_k: torch.Tensor
    cache_v: torch.Tensor
    kv_len: torch.Tensor
    extra: dict = field(default_factory=dict)


def make_decode_batch(w: Workload, B: Optional[int] = None, len_lo: Optional[int] = None,
                      len_hi: Optional[int] = None, Lmax: Optional[int] = None,
                      seed: Optional[int] = None, poison_tail: bool = True) -> DecodeBatch:
    B = w.decode_B if B is None else B
    lo = w.decode_len_lo if len_lo is None else len_lo
    hi = w.decode_len_hi if len_hi is None else len_hi
    Lmax = w.decode_Lmax if Lmax is None else Lmax
    gen = torch.Generator().manual_seed(w.seed if seed is None else seed)
    kv_len = torch.randint(lo, hi + 1, (B,), generator=gen, dtype=torch.int64).to(torch.int32)
    q = _randn_bf16((B, w.Hq, w.D), gen, w.value_scale)
    cache_k = _randn_bf16((B, w.Hkv, Lmax, w.D), gen, w.value_scale)
    cache_v = _randn_bf16((B, w.Hkv, Lmax, w.D), gen, w.value_scale)
    if poison_tail:
        t = torch.arange(Lmax).view(1, 1, Lmax, 1)
        dead = t >= kv_len.view(B, 1, 1, 1).to(torch.int64)
        nan = nan_like((1,))
        cache_k = torch.where(dead, nan, cache_k)
        cache_v = torch.where(dead, nan, cache_v)
    return DecodeBatch(w, q, cache_k.contiguous(), cache_v.contiguous(), kv_len)


def prefill_flops(Hq: int, D: int, seq_lens) -> int:
    """Algorithmic work of causal prefill: 4*D flop per (query, key <= query) pair per query head."""
    return sum(4 * D * Hq * (int(L) * (int(L) + 1) // 2) for L in seq_lens)


def decode_kv_bytes(Hkv: int, D: int, kv_lens) -> int:
    """Algorithmic traffic of decode: K and V of every cached token read once (bf16)."""
    return sum(int(L) * 2 * Hkv * D * 2 for L in kv_lens)


def make_rope_tables(n_pos: int, D: int, base: float = 10000.0):
    """cos / sin tables [n_pos, D/2] (float32) of angle P * base^(-2i/D): inputs of the rotary step, computed
    in float64 and rounded once, as the models' rotary-embedding module hands them to the attention module."""
    import numpy as np

    inv_freq = base ** (-np.arange(0, D, 2, dtype=np.float64) / D)
    ang = np.arange(n_pos, dtype=np.float64)[:, None] * inv_freq[None, :]
    return torch.from_numpy(np.cos(ang).astype(np.float32)), torch.from_numpy(np.sin(ang).astype(np.float32))

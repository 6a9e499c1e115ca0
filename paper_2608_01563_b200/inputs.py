"""Seeded synthetic attention inputs shaped like transformer workloads.

This module holds shapes and random draws only -- none of the attention
arithmetic -- so both the CUDA tests and the CPU oracle tests can share it.

Recipe: for workload number ``c`` (1-based) and sweep index ``s`` the generator is
``torch.Generator("cpu").manual_seed(20260801 + 100*c + s)``; Q, K, V, dO are
drawn in that order with ``torch.randn`` in float32; ``qkv_std`` multiplies
Q, K, V after sampling; for the outlier workloads two Bernoulli(``outlier_p``)
masks (for Q, then K) are drawn with ``torch.rand`` and the selected entries are
multiplied by ``outlier_mul``.  bf16 inputs are the float32 draw rounded to
nearest-even.  Everything is generated on the host.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Tuple

import torch

BASE_SEED = 20260801


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    number: int          # 1-based workload number (enters the seed)
    sweep: int           # sweep index (enters the seed)
    B: int
    H: int
    S: int
    D: int
    causal: bool
    qkv_std: float = 1.0
    outlier_p: float = 0.0
    outlier_mul: float = 1.0

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.D)

    @property
    def seed(self) -> int:
        return BASE_SEED + 100 * self.number + self.sweep

    @property
    def BH(self) -> int:
        return self.B * self.H


def _sweep(idx: int, S: int) -> Workload:
    return Workload(f"decoder_sweep_S{S}", 5, idx, 4, 32, S, 128, True,
                    outlier_p=0.01, outlier_mul=8.0)


WORKLOADS: Dict[str, Workload] = {
    w.name: w
    for w in [
        Workload("tiny", 1, 0, 1, 2, 64, 32, False),
        Workload("gpt2_small", 2, 0, 8, 12, 1024, 64, True, qkv_std=0.5),
        Workload("vit_b_ragged", 3, 0, 32, 12, 197, 64, False),
        Workload("long_context", 4, 0, 2, 16, 4096, 128, True),
        _sweep(0, 512), _sweep(1, 1024), _sweep(2, 2048), _sweep(3, 8192),
    ]
}


def make_inputs(w: Workload, dtype: torch.dtype = torch.float32,
                heads: int | None = None) -> Tuple[torch.Tensor, ...]:
    """Host tensors (Q, K, V, dO), each ``[B,H,S,D]`` in ``dtype``.

    ``heads`` (optional) keeps only the first ``heads`` (b,h) slices, returned as
    ``[1,heads,S,D]``: the full draw is still made so values do not depend on it.
    """
    g = torch.Generator(device="cpu").manual_seed(w.seed)
    shape = (w.B, w.H, w.S, w.D)
    q = torch.randn(shape, generator=g, dtype=torch.float32)
    k = torch.randn(shape, generator=g, dtype=torch.float32)
    v = torch.randn(shape, generator=g, dtype=torch.float32)
    d_o = torch.randn(shape, generator=g, dtype=torch.float32)
    if w.qkv_std != 1.0:
        q *= w.qkv_std
        k *= w.qkv_std
        v *= w.qkv_std
    if w.outlier_p > 0.0:
        mq = torch.rand(shape, generator=g) < w.outlier_p
        mk = torch.rand(shape, generator=g) < w.outlier_p
        q[mq] *= w.outlier_mul
        k[mk] *= w.outlier_mul
    out = []
    for t in (q, k, v, d_o):
        if heads is not None:
            t = t.reshape(1, w.B * w.H, w.S, w.D)[:, :heads].contiguous()
        out.append(t.to(dtype).contiguous())
    return tuple(out)


def random_inputs(seed: int, B: int, H: int, S: int, D: int,
                  dtype: torch.dtype = torch.float32, std: float = 1.0):
    """Plain N(0, std^2) Q, K, V, dO for edge-shape tests."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    return tuple(
        (torch.randn((B, H, S, D), generator=g, dtype=torch.float32) * std).to(dtype).contiguous()
        for _ in range(4)
    )


# ---------------------------------------------------------------------------------------------
# Cross-attention and grouped key/value heads: q, dO are [B,H,Sq,D]; k, v are [B,Hkv,Sk,D].
@dataclasses.dataclass(frozen=True)
class ExtWorkload:
    name: str
    number: int          # enters the seed like Workload.number
    B: int
    H: int
    Hkv: int
    Sq: int
    Sk: int
    D: int
    causal: bool

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.D)

    @property
    def seed(self) -> int:
        return BASE_SEED + 100 * self.number

    @property
    def pairs(self) -> float:
        """Score pairs per (batch, query head), counted like the square workloads: a causal
        triangle of side Sq counts Sq^2/2, the rectangle of always-visible keys in front of it fully."""
        return self.Sq * (self.Sk - self.Sq) + self.Sq * self.Sq / 2.0 if self.causal else float(self.Sq * self.Sk)


EXT_WORKLOADS: Dict[str, ExtWorkload] = {
    w.name: w
    for w in [
        # decoder block with grouped key/value heads at the size of the decoder sweep (S = 2048)
        ExtWorkload("gqa_decoder", 6, 4, 32, 8, 2048, 2048, 128, True),
        # text cross-attention of a latent-diffusion U-Net: a 32x32 latent (1024 queries) over 77 text tokens
        ExtWorkload("cross_attn_text", 7, 16, 8, 8, 1024, 77, 64, False),
        # action tokens over vision-language context tokens, batched
        ExtWorkload("cross_attn_action", 8, 64, 8, 8, 50, 16, 64, False),
        # chunked causal continuation: 512 new queries at the end of a 4096-token context, grouped heads
        ExtWorkload("gqa_suffix", 9, 2, 16, 4, 512, 4096, 128, True),
    ]
}


def make_inputs_ext(w: ExtWorkload, dtype: torch.dtype = torch.float32) -> Tuple[torch.Tensor, ...]:
    """Host tensors (Q [B,H,Sq,D], K, V [B,Hkv,Sk,D], dO [B,H,Sq,D]) ~ N(0,1), drawn in that order
    with ``torch.randn`` in float32 from ``torch.Generator("cpu").manual_seed(w.seed)``."""
    g = torch.Generator(device="cpu").manual_seed(w.seed)
    q = torch.randn((w.B, w.H, w.Sq, w.D), generator=g, dtype=torch.float32)
    k = torch.randn((w.B, w.Hkv, w.Sk, w.D), generator=g, dtype=torch.float32)
    v = torch.randn((w.B, w.Hkv, w.Sk, w.D), generator=g, dtype=torch.float32)
    d_o = torch.randn((w.B, w.H, w.Sq, w.D), generator=g, dtype=torch.float32)
    return tuple(t.to(dtype).contiguous() for t in (q, k, v, d_o))

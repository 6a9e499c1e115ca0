"""Seeded random shapes through every entry point, both modes, against the f64 oracle.
The fixed-shape files cover the edges deliberately; this one guards against shape combinations
nobody thought of (lengths around tile multiples, head groups, offsets)."""
import math
import random

import pytest
import torch

from paper_2608_01563_b200 import binding as mgn
from paper_2608_01563_b200 import inputs as synth

import helpers as hp

pytestmark = pytest.mark.gpu


def _shapes(seed, n, fast):
    rnd = random.Random(seed)
    out = []
    for _ in range(n):
        D = rnd.choice([64, 128] if fast else [32, 64, 128])
        Hkv = rnd.choice([1, 2, 3])
        G = rnd.choice([1, 1, 2, 4])
        B = rnd.choice([1, 2])
        base = rnd.choice([1, 17, 64, 128, 129, 191, 256, 300, 385, 512])
        Sq = max(1, base + rnd.randint(-3, 3))
        causal = rnd.random() < 0.5
        if rnd.random() < 0.5:
            Sk = Sq
        else:
            Sk = max(1, rnd.choice([16, 77, 130, 260, 400, 640]) + rnd.randint(-2, 2))
        if causal and Sq > Sk:
            Sq, Sk = Sk, Sq
        out.append((B, Hkv * G, Hkv, Sq, Sk, D, causal))
    return out


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal", _shapes(20260803, 24, fast=False))
def test_strict_random_shapes(B, H, Hkv, Sq, Sk, D, causal):
    scale = 1.0 / math.sqrt(D)
    q, _, _, d_o = synth.random_inputs(900, B, H, Sq, D)
    _, k, v, _ = synth.random_inputs(901, B, Hkv, Sk, D)
    got = hp.run_cuda_ext(q, k, v, d_o, causal, scale, mgn.MODE_STRICT_F32)
    ref = hp.run_oracle_ext(q, k, v, d_o, causal, scale)
    hp.check_strict(got, ref, literal_max_abs=False, label=f"random strict {B,H,Hkv,Sq,Sk,D,causal} ")


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal", _shapes(20260804, 24, fast=True))
def test_fast_random_shapes(B, H, Hkv, Sq, Sk, D, causal):
    scale = 1.0 / math.sqrt(D)
    q, _, _, d_o = synth.random_inputs(902, B, H, Sq, D, dtype=torch.bfloat16)
    _, k, v, _ = synth.random_inputs(903, B, Hkv, Sk, D, dtype=torch.bfloat16)
    got = hp.run_cuda_ext(q, k, v, d_o, causal, scale, mgn.MODE_FAST_BF16)
    ref = hp.run_oracle_ext(q, k, v, d_o, causal, scale)
    hp.check_fast(got, ref, label=f"random fast {B,H,Hkv,Sq,Sk,D,causal} ")

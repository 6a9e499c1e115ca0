"""Deterministic backward (mgn_attn_bwd_deterministic), both modes: fused dK+dV kernel without the dQ
product and reductions, plus a separate dQ pass.  Checked element by element against the f64 oracle,
and for bit-identical results across runs."""
import math

import pytest
import torch

from paper_2608_01563_b200 import binding as mgn
from paper_2608_01563_b200 import inputs as synth

import helpers as hp

pytestmark = pytest.mark.gpu
MODE = mgn.MODE_STRICT_F32


def _run(q, k, v, d_o, causal, scale, mode=MODE):
    dev = "cuda"
    B, H, Sq, D = q.shape
    _, Hkv, Sk, _ = k.shape
    qd, kd, vd, dod = (t.to(dev) for t in (q, k, v, d_o))
    o = torch.empty_like(qd)
    lse = torch.empty(B, H, Sq, device=dev)
    mgn.mgn_attn_fwd_ext(qd, kd, vd, o, lse, causal, scale, mode)
    dq = hp.Guarded((B, H, Sq, D), q.dtype)
    dk, dv = (hp.Guarded((B, Hkv, Sk, D), q.dtype) for _ in range(2))
    ws = mgn.alloc_workspace(B, H, Sq, D, mode)
    ws.fill_(0xFF)
    mgn.mgn_attn_bwd_deterministic(qd, kd, vd, o, dod, lse, dq.view, dk.view, dv.view, ws, causal, scale, mode)
    mgn.mgn_attn_check()
    return {"dQ": dq.check("dQ"), "dK": dk.check("dK"), "dV": dv.check("dV")}


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal", [
    (1, 2, 2, 64, 64, 32, False),
    (2, 3, 3, 197, 197, 64, False),
    (1, 4, 4, 300, 300, 64, True),
    (1, 2, 2, 257, 257, 128, True),
    (1, 1, 1, 1, 1, 64, True),
    (2, 8, 2, 130, 130, 64, True),       # grouped heads
    (1, 8, 8, 50, 16, 64, False),        # cross-attention
    (1, 4, 2, 100, 260, 128, True),      # bottom-right causal with grouped heads
])
def test_matches_oracle(B, H, Hkv, Sq, Sk, D, causal):
    scale = 1.0 / math.sqrt(D)
    q, _, _, d_o = synth.random_inputs(700, B, H, Sq, D)
    _, k, v, _ = synth.random_inputs(701, B, Hkv, Sk, D)
    got = {n: t.double().numpy() for n, t in _run(q, k, v, d_o, causal, scale).items()}
    ref = hp.run_oracle_ext(q, k, v, d_o, causal, scale)
    hp.check_strict(got, ref, names=("dQ", "dK", "dV"), literal_max_abs=False,
                    label=f"deterministic {B,H,Hkv,Sq,Sk,D,causal} ")


def test_results_are_bit_identical_across_runs():
    w = synth.WORKLOADS["gpt2_small"]
    q, k, v, d_o = synth.make_inputs(w, heads=24)
    a = _run(q, k, v, d_o, w.causal, w.scale)
    b = _run(q, k, v, d_o, w.causal, w.scale)
    c = _run(q, k, v, d_o, w.causal, w.scale)
    for n in ("dQ", "dK", "dV"):
        assert torch.equal(a[n], b[n]) and torch.equal(a[n], c[n]), f"{n} differs between runs"


def test_gpt2_small_heads_match_oracle():
    w = synth.WORKLOADS["gpt2_small"]
    q, k, v, d_o = synth.make_inputs(w, heads=6)
    got = {n: t.double().numpy() for n, t in _run(q, k, v, d_o, w.causal, w.scale).items()}
    ref = hp.run_oracle_ext(q, k, v, d_o, w.causal, w.scale)
    hp.check_strict(got, ref, names=("dQ", "dK", "dV"), literal_max_abs=False, label="deterministic gpt2_small ")


FAST = mgn.MODE_FAST_BF16
BF = torch.bfloat16


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal", [
    (1, 2, 2, 64, 64, 64, False),
    (2, 3, 3, 197, 197, 64, False),
    (1, 4, 4, 300, 300, 64, True),
    (1, 2, 2, 257, 257, 128, True),
    (1, 1, 1, 1, 1, 64, True),
    (2, 8, 2, 130, 130, 128, True),      # grouped heads
    (1, 8, 8, 50, 16, 64, False),        # cross-attention
    (1, 4, 2, 100, 260, 128, True),      # bottom-right causal with grouped heads
    (1, 4, 4, 520, 520, 128, False),     # several key blocks per query tile
])
def test_fast_matches_oracle(B, H, Hkv, Sq, Sk, D, causal):
    scale = 1.0 / math.sqrt(D)
    q, _, _, d_o = synth.random_inputs(710, B, H, Sq, D, dtype=BF)
    _, k, v, _ = synth.random_inputs(711, B, Hkv, Sk, D, dtype=BF)
    got = {n: t.double().numpy() for n, t in _run(q, k, v, d_o, causal, scale, FAST).items()}
    ref = hp.run_oracle_ext(q, k, v, d_o, causal, scale)
    hp.check_fast(got, ref, names=("dQ", "dK", "dV"), label=f"deterministic fast {B,H,Hkv,Sq,Sk,D,causal} ")


def test_fast_results_are_bit_identical_across_runs():
    w = synth.WORKLOADS["long_context"]
    q, k, v, d_o = synth.make_inputs(w, dtype=BF, heads=8)
    a = _run(q, k, v, d_o, w.causal, w.scale, FAST)
    b = _run(q, k, v, d_o, w.causal, w.scale, FAST)
    c = _run(q, k, v, d_o, w.causal, w.scale, FAST)
    for n in ("dQ", "dK", "dV"):
        assert torch.equal(a[n], b[n]) and torch.equal(a[n], c[n]), f"{n} differs between runs"


def test_fast_long_context_heads_match_oracle():
    w = synth.WORKLOADS["long_context"]
    q, k, v, d_o = synth.make_inputs(w, dtype=BF, heads=3)
    got = {n: t.double().numpy() for n, t in _run(q, k, v, d_o, w.causal, w.scale, FAST).items()}
    ref = hp.run_oracle_ext(q, k, v, d_o, w.causal, w.scale)
    hp.check_fast(got, ref, names=("dQ", "dK", "dV"), label="deterministic fast long_context ")

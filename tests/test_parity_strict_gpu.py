"""Strict (f32 FFMA) mode: CUDA path vs the f64 oracle, element by element, through the C ABI."""
import math

import numpy as np
import pytest
import torch

from paper_2608_01563_b200 import binding as mgn
from paper_2608_01563_b200 import inputs as synth

import helpers as hp

pytestmark = pytest.mark.gpu
MODE = mgn.MODE_STRICT_F32


def _full_parity(w, heads=None, literal=True):
    q, k, v, d_o = synth.make_inputs(w)
    res = hp.run_cuda(q, k, v, d_o, w.causal, w.scale, MODE)
    ref = hp.run_oracle(q, k, v, d_o, w.causal, w.scale, heads)
    got = hp.select(res, w.B, w.H, heads)
    rep = hp.check_strict(got, ref, literal_max_abs=literal, label=w.name + " ")
    hp.check_invariants(q, k, v, d_o, res, rtol=2e-5)
    return rep


def test_tiny_all_heads():
    _full_parity(synth.WORKLOADS["tiny"])


def test_gpt2_small_shaped_causal_all_heads():
    _full_parity(synth.WORKLOADS["gpt2_small"])


def test_vit_b_shaped_ragged_all_heads():
    _full_parity(synth.WORKLOADS["vit_b_ragged"])


@pytest.mark.parametrize("name,heads", [
    ("decoder_sweep_S512", [0, 37, 90, 127]),
    ("decoder_sweep_S1024", [0, 127]),
    ("decoder_sweep_S2048", [64]),
])
def test_decoder_sweep_outliers_head_subset(name, heads):
    # Scores reach +-64 here and |dQ|,|dK| reach tens: the absolute bound is applied
    # relative to max(1, max|ref|); rel-L2 is the literal gate.
    _full_parity(synth.WORKLOADS[name], heads=heads, literal=False)


def test_decoder_sweep_longest_sequence_two_heads():
    """S = 8192 (the largest configured size), in the launch configuration the benchmark times:
    two heads element by element against the oracle, invariants on 16 heads."""
    w = synth.WORKLOADS["decoder_sweep_S8192"]
    heads = [5, 100]
    q, k, v, d_o = synth.make_inputs(w)
    res = hp.run_cuda(q, k, v, d_o, w.causal, w.scale, MODE)
    ref = hp.run_oracle(q, k, v, d_o, w.causal, w.scale, heads)
    hp.check_strict(hp.select(res, w.B, w.H, heads), ref, literal_max_abs=False, label=w.name + " ")
    hp.check_invariants(q, k, v, d_o, res, rtol=2e-5, max_heads=16)


@pytest.mark.parametrize("D", [32, 64, 128])
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("S", [1, 2, 63, 64, 65, 127, 129, 197, 300])
def test_edge_shapes(S, D, causal):
    B, H = 1, 3
    q, k, v, d_o = synth.random_inputs(1000 + S + D, B, H, S, D)
    scale = 1.0 / math.sqrt(D)
    res = hp.run_cuda(q, k, v, d_o, causal, scale, MODE)
    ref = hp.run_oracle(q, k, v, d_o, causal, scale)
    hp.check_strict(hp.select(res, B, H), ref, label=f"S={S} D={D} causal={causal} ")


@pytest.mark.parametrize("scale", [0.0, -0.3, 2.0])
def test_unusual_scales(scale):
    B, H, S, D = 2, 2, 150, 64
    q, k, v, d_o = synth.random_inputs(77, B, H, S, D, std=0.7)
    res = hp.run_cuda(q, k, v, d_o, True, scale, MODE)
    ref = hp.run_oracle(q, k, v, d_o, True, scale)
    # scale 2.0 drives |dQ|,|dK| to tens, so the absolute bound is taken relative to max(1, max|ref|)
    hp.check_strict(hp.select(res, B, H), ref, literal_max_abs=False, label=f"scale={scale} ")


def test_backward_accepts_given_o_and_lse():
    """Backward in isolation: feed the oracle's O and LSE rounded to f32."""
    B, H, S, D = 1, 2, 200, 64
    q, k, v, d_o = synth.random_inputs(5, B, H, S, D)
    scale = 0.125
    ref = hp.run_oracle(q, k, v, d_o, False, scale)
    o32 = torch.from_numpy(ref["O"]).float().reshape(B, H, S, D)
    l32 = torch.from_numpy(ref["LSE"]).float().reshape(B, H, S)
    res = hp.run_cuda(q, k, v, d_o, False, scale, MODE, given_o=o32, given_lse=l32)
    hp.check_strict(hp.select(res, B, H), ref)


def test_determinism_and_atomic_dq():
    w = synth.WORKLOADS["vit_b_ragged"]
    q, k, v, d_o = synth.make_inputs(w, heads=24)
    a = hp.run_cuda(q, k, v, d_o, False, w.scale, MODE)
    b = hp.run_cuda(q, k, v, d_o, False, w.scale, MODE)
    for n in ("O", "LSE", "dK", "dV"):
        assert torch.equal(a[n], b[n]), f"{n} differs between two runs"
    assert hp.rel_l2(a["dQ"].double().numpy(), b["dQ"].double().numpy()) <= 1e-6


def test_runs_on_a_side_stream_without_host_sync():
    B, H, S, D = 2, 4, 260, 64
    q, k, v, d_o = synth.random_inputs(9, B, H, S, D)
    scale = 0.125
    st = torch.cuda.Stream()
    qd, kd, vd, dod = (t.cuda() for t in (q, k, v, d_o))
    o = torch.empty_like(qd); lse = torch.empty(B, H, S, device="cuda")
    dq, dk, dv = (torch.empty_like(qd) for _ in range(3))
    ws = mgn.alloc_workspace(B, H, S, D, MODE)
    torch.cuda.synchronize()
    with torch.cuda.stream(st):
        big = torch.randn(4096, 4096, device="cuda")
        for _ in range(10):
            big = big @ big * 1e-3          # keeps the stream busy ahead of the calls
        mgn.mgn_attn_fwd(qd, kd, vd, o, lse, True, scale, MODE)
        mgn.mgn_attn_bwd(qd, kd, vd, o, dod, lse, dq, dk, dv, ws, True, scale, MODE)
    st.synchronize()
    mgn.mgn_attn_check(st.cuda_stream)
    ref = hp.run_oracle(q, k, v, d_o, True, scale)
    got = hp.select({"O": o.cpu(), "LSE": lse.cpu(), "dQ": dq.cpu(), "dK": dk.cpu(), "dV": dv.cpu()}, B, H)
    hp.check_strict(got, ref)


def test_misuse_is_reported_not_executed():
    q = torch.zeros(1, 1, 8, 64, device="cuda")
    lse = torch.zeros(1, 1, 8, device="cuda")
    with pytest.raises(mgn.MgnError) as e:
        mgn.mgn_attn_fwd(q, q, q, q, lse, True, float("nan"), MODE)
    assert e.value.status == 1
    q48 = torch.zeros(1, 1, 8, 48, device="cuda")
    with pytest.raises(mgn.MgnError) as e:
        mgn.mgn_attn_fwd(q48, q48, q48, q48, lse, True, 1.0, MODE)
    assert e.value.status == 2

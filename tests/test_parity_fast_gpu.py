"""Fast (bf16 tensor-core) mode: CUDA path vs the f64 oracle through the C ABI.

The oracle receives the bf16-rounded inputs (exact in f64), so input quantisation is not
counted as error; rounding of P, dS and of the bf16 outputs is.  Gate: rel-L2 <= 2e-2."""
import math

import numpy as np
import pytest
import torch

from paper_2608_01563_b200 import binding as mgn
from paper_2608_01563_b200 import inputs as synth

import helpers as hp

pytestmark = pytest.mark.gpu
MODE = mgn.MODE_FAST_BF16
BF = torch.bfloat16


@pytest.mark.parametrize("D", [32, 64, 128])
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("S", [1, 2, 63, 64, 65, 127, 128, 129, 197, 256, 257, 300, 520])
def test_forward_edge_shapes(S, D, causal):
    B, H = 1, 3
    q, k, v, d_o = synth.random_inputs(2000 + S + D, B, H, S, D, dtype=BF)
    scale = 1.0 / math.sqrt(D)
    res = hp.run_cuda(q, k, v, d_o, causal, scale, MODE, run_bwd=False)
    ref = hp.run_oracle(q, k, v, d_o, causal, scale)
    hp.check_fast(hp.select(res, B, H), ref, names=("O",), label=f"S={S} D={D} causal={causal} ")


@pytest.mark.parametrize("D", [32, 64, 128])
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("S", [1, 2, 63, 64, 65, 127, 128, 129, 197, 256, 257, 300, 520])
def test_forward_backward_edge_shapes(S, D, causal):
    B, H = 1, 3
    q, k, v, d_o = synth.random_inputs(3000 + S + D, B, H, S, D, dtype=BF)
    scale = 1.0 / math.sqrt(D)
    res = hp.run_cuda(q, k, v, d_o, causal, scale, MODE)
    ref = hp.run_oracle(q, k, v, d_o, causal, scale)
    hp.check_fast(hp.select(res, B, H), ref, label=f"S={S} D={D} causal={causal} ")


@pytest.mark.parametrize("order", [0, 1])
@pytest.mark.parametrize("B,H,S,D,causal", [
    (1, 3, 300, 64, True),       # ragged tail, odd number of blocks, fewer items than CTAs
    (2, 40, 700, 128, True),     # several items per CTA, odd number of key blocks and of tile pairs
    (2, 40, 640, 128, False),    # non-causal: equal weights
    (1, 150, 257, 64, True),     # one more item pair than CTAs can share evenly
])
def test_both_item_orders_match_the_oracle(order, B, H, S, D, causal):
    """The two work-item orders of the persistent kernels (block-major and head-major) visit the
    same items; both are forced here at sizes where the default would pick only one of them."""
    scale = 1.0 / math.sqrt(D)
    q, k, v, d_o = synth.random_inputs(77 + order, B, H, S, D, dtype=BF)
    heads = sorted({0, (B * H) // 2, B * H - 1})
    mgn.mgn_attn_fast_item_order(order)
    try:
        res = hp.run_cuda(q, k, v, d_o, causal, scale, MODE)
    finally:
        mgn.mgn_attn_fast_item_order(-1)
    ref = hp.run_oracle(q, k, v, d_o, causal, scale, heads)
    hp.check_fast(hp.select(res, B, H, heads), ref, label=f"order={order} ")
    hp.check_invariants(q, k, v, d_o, res, rtol=2e-2)


def test_forward_large_max_growth_triggers_rescale():
    """Keys grow along the sequence so the running maximum moves by far more than the lazy threshold."""
    B, H, S, D = 1, 2, 1024, 128
    q, k, v, d_o = synth.random_inputs(11, B, H, S, D, dtype=torch.float32)
    ramp = torch.linspace(0.1, 3.0, S).view(1, 1, S, 1)
    k = (k * ramp).to(BF)
    q, v, d_o = q.to(BF), v.to(BF), d_o.to(BF)
    for causal in (False, True):
        res = hp.run_cuda(q, k, v, d_o, causal, 0.3, MODE, run_bwd=False)
        ref = hp.run_oracle(q, k, v, d_o, causal, 0.3)
        hp.check_fast(hp.select(res, B, H), ref, names=("O",))


@pytest.mark.parametrize("causal", [False, True])
def test_forward_stepwise_growth_moves_the_reference_point_in_every_block(causal):
    """Every query has 4 and key block b has 25 b in component 0, so with scale 0.5 the scores of a
    row jump by 50 (72 in the log2 domain) from each 128-key block to the next: more than the growth
    limit of the pass (2^60), so every block takes the redo path (find the maxima, rescale O and l,
    repeat the pass).  O and the saved log-sum-exp must still match."""
    B, H, S, D = 1, 2, 1152, 128
    q, k, v, d_o = synth.random_inputs(13, B, H, S, D, dtype=torch.float32)
    q[..., 0] = 4.0
    k[..., 0] = (25.0 * (torch.arange(S) // 128)).view(1, 1, S)
    q, k, v, d_o = q.to(BF), k.to(BF), v.to(BF), d_o.to(BF)
    res = hp.run_cuda(q, k, v, d_o, causal, 0.5, MODE, run_bwd=False)
    ref = hp.run_oracle(q, k, v, d_o, causal, 0.5)
    got = hp.select(res, B, H)
    hp.check_fast(got, ref, names=("O",), label="stepwise growth ")
    err = np.abs(got["LSE"] - ref["LSE"])
    assert (err <= 2e-2 + 1e-3 * np.abs(ref["LSE"])).all(), f"LSE off by up to {err.max()}"


@pytest.mark.parametrize("D,causal", [(128, False), (128, True), (64, True)])
def test_forward_heavy_tailed_scores_below_the_growth_limit(D, causal):
    """1 % of Q and K scaled by 8 (the decoder sweep's distribution) at a length of several blocks:
    the reference point of a row stays where the first block put it although later scores are far
    larger (p up to about 2^40); O and LSE must match."""
    B, H, S = 1, 2, 1024
    q, k, v, d_o = synth.random_inputs(14, B, H, S, D, dtype=torch.float32)
    g = torch.Generator().manual_seed(15)
    q = torch.where(torch.rand(q.shape, generator=g) < 0.01, 8.0 * q, q)
    k = torch.where(torch.rand(k.shape, generator=g) < 0.01, 8.0 * k, k)
    k[:, :, :128] *= 0.05                       # the first block sets a low reference point
    q, k, v, d_o = q.to(BF), k.to(BF), v.to(BF), d_o.to(BF)
    res = hp.run_cuda(q, k, v, d_o, causal, 0.5, MODE, run_bwd=False)
    ref = hp.run_oracle(q, k, v, d_o, causal, 0.5)
    got = hp.select(res, B, H)
    hp.check_fast(got, ref, names=("O",), label="heavy tails ")
    err = np.abs(got["LSE"] - ref["LSE"])
    assert (err <= 2e-2 + 1e-3 * np.abs(ref["LSE"])).all(), f"LSE off by up to {err.max()}"


@pytest.mark.parametrize("scale", [0.0, -0.2])
def test_forward_unusual_scales(scale):
    B, H, S, D = 1, 2, 300, 64
    q, k, v, d_o = synth.random_inputs(12, B, H, S, D, dtype=BF)
    res = hp.run_cuda(q, k, v, d_o, True, scale, MODE, run_bwd=False)
    ref = hp.run_oracle(q, k, v, d_o, True, scale)
    hp.check_fast(hp.select(res, B, H), ref, names=("O",))


def _workload_parity(name, heads):
    w = synth.WORKLOADS[name]
    q, k, v, d_o = synth.make_inputs(w, dtype=BF)
    res = hp.run_cuda(q, k, v, d_o, w.causal, w.scale, MODE)
    ref = hp.run_oracle(q, k, v, d_o, w.causal, w.scale, heads)
    rep = hp.check_fast(hp.select(res, w.B, w.H, heads), ref, label=name + " ")
    hp.check_invariants(q, k, v, d_o, res, rtol=2e-2)
    return rep


def test_long_context_all_heads():
    _workload_parity("long_context", None)


@pytest.mark.parametrize("name,heads", [
    ("decoder_sweep_S512", [0, 37, 127]),
    ("decoder_sweep_S1024", [0, 127]),
    ("decoder_sweep_S2048", [64]),
])
def test_decoder_sweep_head_subset(name, heads):
    _workload_parity(name, heads)


def test_decoder_sweep_longest_sequence_two_heads():
    w = synth.WORKLOADS["decoder_sweep_S8192"]
    heads = [5, 100]
    q, k, v, d_o = synth.make_inputs(w, dtype=BF)
    res = hp.run_cuda(q, k, v, d_o, w.causal, w.scale, MODE)
    ref = hp.run_oracle(q, k, v, d_o, w.causal, w.scale, heads)
    hp.check_fast(hp.select(res, w.B, w.H, heads), ref, label=w.name + " ")
    hp.check_invariants(q, k, v, d_o, res, rtol=2e-2, max_heads=16)


@pytest.mark.parametrize("order", [0, 1])
def test_head_size_32_several_items_per_cta(order):
    """Head size 32 (run as a zero-padded 64-wide problem) at a size with several work items per
    CTA, under both extremes of the work-item list, and through the deterministic backward."""
    B, H, S, D, causal = 2, 80, 700, 32, True
    scale = 1.0 / math.sqrt(D)
    q, k, v, d_o = synth.random_inputs(91 + order, B, H, S, D, dtype=BF)
    heads = [0, 77, B * H - 1]
    mgn.mgn_attn_fast_item_order(order)
    try:
        res = hp.run_cuda(q, k, v, d_o, causal, scale, MODE)
    finally:
        mgn.mgn_attn_fast_item_order(-1)
    ref = hp.run_oracle(q, k, v, d_o, causal, scale, heads)
    hp.check_fast(hp.select(res, B, H, heads), ref, label=f"D=32 order={order} ")
    hp.check_invariants(q, k, v, d_o, res, rtol=2e-2)
    qd, kd, vd, dod = (t.cuda() for t in (q, k, v, d_o))
    dq, dk, dv = (torch.full_like(qd, float("nan")) for _ in range(3))
    ws = mgn.alloc_workspace(B, H, S, D, MODE)
    mgn.mgn_attn_bwd_deterministic(qd, kd, vd, res["O"].cuda(), dod, res["LSE"].cuda(), dq, dk, dv, ws, causal, scale, MODE)
    mgn.mgn_attn_check()
    det = hp.select({"dQ": dq.cpu(), "dK": dk.cpu(), "dV": dv.cpu()}, B, H, heads)
    hp.check_fast(det, ref, names=("dQ", "dK", "dV"), label="D=32 deterministic ")

"""Output projection fused with attention at its two seams (fast mode): CUDA path through the C ABI
against the f64 oracle, element by element.  The oracle receives the bf16-rounded inputs; gate: the
fast mode's rel-L2 <= 2e-2 (measured a few 1e-3: bf16 output rounding)."""
import math

import numpy as np
import pytest
import torch

from oracle import attn_oracle as orc
from paper_2608_01563_b200 import binding as mgn
from paper_2608_01563_b200 import inputs as synth

import helpers as hp

pytestmark = pytest.mark.gpu
MODE = mgn.MODE_FAST_BF16
BF = torch.bfloat16

SHAPES = [
    # B, H, S, D, E
    (1, 2, 128, 128, 256),        # one tile exactly
    (2, 3, 197, 64, 200),         # ragged rows, E not a tile multiple, H*D not a multiple of 256
    (1, 5, 300, 128, 640),        # several column tiles, odd head count
    (3, 4, 1, 64, 8),             # a single position, the smallest E
    (2, 16, 520, 128, 2048),      # many contraction slices (K = 2048), several row tiles
]


def _draw(seed, B, H, S, D, E):
    g = torch.Generator().manual_seed(seed)
    o = torch.randn(B, H, S, D, generator=g).to(BF)
    w = (torch.randn(H * D, E, generator=g) / math.sqrt(H * D)).to(BF)
    d_y = torch.randn(B, S, E, generator=g).to(BF)
    return o, w, d_y


@pytest.mark.parametrize("B,H,S,D,E", SHAPES)
def test_forward_projection_reads_head_major_o(B, H, S, D, E):
    o, w, _ = _draw(10 + S, B, H, S, D, E)
    y = hp.Guarded((B, S, E), BF)
    mgn.mgn_out_proj_fwd(o.cuda(), w.cuda(), y.view, MODE)
    mgn.mgn_attn_check()
    got = y.check("Y").double().numpy()
    ref = orc.out_proj_fwd(o.double().numpy(), w.double().numpy())
    assert hp.rel_l2(got, ref) <= hp.FAST_REL_L2, hp.rel_l2(got, ref)


@pytest.mark.parametrize("B,H,S,D,E", SHAPES)
def test_do_producer_writes_do_and_delta(B, H, S, D, E):
    o, w, d_y = _draw(20 + S, B, H, S, D, E)
    d_o = hp.Guarded((B, H, S, D), BF)
    delta = hp.Guarded((B, H, S), torch.float32)
    mgn.mgn_out_proj_bwd_data(d_y.cuda(), w.cuda(), o.cuda(), d_o.view, delta.view, MODE)
    mgn.mgn_attn_check()
    got_do = d_o.check("dO").double().numpy()
    got_dl = delta.check("delta").double().numpy()
    ref_do, ref_dl, _ = orc.out_proj_bwd(d_y.double().numpy(), w.double().numpy(), o.double().numpy())
    assert hp.rel_l2(got_do, ref_do) <= hp.FAST_REL_L2
    assert hp.rel_l2(got_dl, ref_dl) <= hp.FAST_REL_L2
    # and delta is exactly the row statistic of the stored (bf16) dO, as the attention backward defines it
    own = (torch.from_numpy(got_do) * o.double()).sum(-1).numpy()
    np.testing.assert_allclose(got_dl, own, rtol=1e-4, atol=1e-4)


@pytest.mark.parametrize("mode,dtype", [(mgn.MODE_FAST_BF16, BF), (mgn.MODE_STRICT_F32, torch.float32)])
@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal", [(2, 4, 4, 300, 300, 64, True), (1, 4, 2, 130, 260, 128, True),
                                                     (2, 2, 2, 77, 200, 64, False)])
def test_backward_with_given_delta_matches_the_oracle(mode, dtype, B, H, Hkv, Sq, Sk, D, causal):
    """mgn_attn_bwd_given_delta with delta = rowsum(dO o O) from the forward's own O."""
    g = torch.Generator().manual_seed(31 + Sq)
    q = torch.randn(B, H, Sq, D, generator=g).to(dtype)
    k = torch.randn(B, Hkv, Sk, D, generator=g).to(dtype)
    v = torch.randn(B, Hkv, Sk, D, generator=g).to(dtype)
    d_o = torch.randn(B, H, Sq, D, generator=g).to(dtype)
    scale = 1.0 / math.sqrt(D)
    qd, kd, vd, dod = (t.cuda() for t in (q, k, v, d_o))
    o = torch.empty_like(qd)
    lse = torch.empty(B, H, Sq, device="cuda")
    mgn.mgn_attn_fwd_ext(qd, kd, vd, o, lse, causal, scale, mode)
    delta = (o.float() * dod.float()).sum(-1).contiguous()
    dq = hp.Guarded((B, H, Sq, D), dtype)
    dk, dv = (hp.Guarded((B, Hkv, Sk, D), dtype) for _ in range(2))
    ws = mgn.alloc_workspace(B, H, Sq, D, mode)
    ws.fill_(0xFF)
    mgn.mgn_attn_bwd_given_delta(qd, kd, vd, dod, lse, delta, dq.view, dk.view, dv.view, ws, causal, scale, mode)
    mgn.mgn_attn_check()
    got = {"dQ": dq.check("dQ").double().numpy(), "dK": dk.check("dK").double().numpy(), "dV": dv.check("dV").double().numpy()}
    ref = hp.run_oracle_ext(q, k, v, d_o, causal, scale)
    if mode == mgn.MODE_STRICT_F32:
        hp.check_strict(got, ref, names=("dQ", "dK", "dV"), label="given delta ")
    else:
        hp.check_fast(got, ref, names=("dQ", "dK", "dV"), label="given delta ")


def test_projection_then_attention_backward_end_to_end():
    """dY -> (dO, delta) by the fused producer -> attention backward without its preprocess pass,
    against the oracle chain on the same bf16 inputs."""
    B, H, S, D, E = 2, 4, 384, 128, 512
    w_att = synth.Workload("proj_chain", 9, 1, B, H, S, D, True)
    q, k, v, _ = synth.make_inputs(w_att, dtype=BF)
    g = torch.Generator().manual_seed(5)
    w = (torch.randn(H * D, E, generator=g) / math.sqrt(H * D)).to(BF)
    d_y = torch.randn(B, S, E, generator=g).to(BF)
    qd, kd, vd = (t.cuda() for t in (q, k, v))
    o = torch.empty_like(qd); lse = torch.empty(B, H, S, device="cuda")
    mgn.mgn_attn_fwd(qd, kd, vd, o, lse, True, w_att.scale, MODE)
    d_o = torch.empty_like(qd); delta = torch.empty(B, H, S, device="cuda")
    mgn.mgn_out_proj_bwd_data(d_y.cuda(), w.cuda(), o, d_o, delta, MODE)
    dq, dk, dv = (torch.empty_like(qd) for _ in range(3))
    ws = mgn.alloc_workspace(B, H, S, D, MODE)
    mgn.mgn_attn_bwd_given_delta(qd, kd, vd, d_o, lse, delta, dq, dk, dv, ws, True, w_att.scale, MODE)
    mgn.mgn_attn_check()
    # oracle chain in f64: O from the attention oracle, dO from the projection oracle, then attention backward
    o_ref, _ = orc.attn_fwd(q.double().numpy(), k.double().numpy(), v.double().numpy(), True, w_att.scale)
    do_ref, _, _ = orc.out_proj_bwd(d_y.double().numpy(), w.double().numpy(), o_ref)
    _, _, dq_r, dk_r, dv_r = orc.attn_bwd(q.double().numpy(), k.double().numpy(), v.double().numpy(), do_ref, True, w_att.scale)
    for name, got, ref in (("dQ", dq, dq_r), ("dK", dk, dk_r), ("dV", dv, dv_r)):
        err = hp.rel_l2(got.double().cpu().numpy(), ref)
        assert err <= hp.FAST_REL_L2, f"{name}: {err:.3e}"


@pytest.mark.parametrize("B,H,S,D,E", SHAPES)
def test_weight_gradient_contracts_over_all_positions(B, H, S, D, E):
    o, w, d_y = _draw(40 + S, B, H, S, D, E)
    d_w = hp.Guarded((H * D, E), BF)
    mgn.mgn_out_proj_bwd_weight(o.cuda(), d_y.cuda(), d_w.view, MODE)
    mgn.mgn_attn_check()
    got = d_w.check("dW").double().numpy()
    _, _, ref = orc.out_proj_bwd(d_y.double().numpy(), w.double().numpy(), o.double().numpy())
    assert hp.rel_l2(got, ref) <= hp.FAST_REL_L2, hp.rel_l2(got, ref)


@pytest.mark.parametrize("B,S,E,H,Hkv,D", [
    (1, 128, 64, 2, 2, 128),       # one tile
    (2, 197, 200, 3, 1, 64),       # ragged rows, E not a slice multiple, (H + 2 Hkv) D not a tile multiple
    (1, 300, 512, 5, 5, 128),      # odd head count: a column tile that mixes key and value heads
    (3, 1, 8, 4, 2, 64),           # a single position
    (2, 520, 1024, 8, 2, 128),     # grouped key/value heads, several row tiles and contraction slices
])
def test_qkv_projection_with_rotary_embedding(B, S, E, H, Hkv, D):
    g = torch.Generator().manual_seed(50 + S)
    x = torch.randn(B, S, E, generator=g).to(BF)
    w = (torch.randn((H + 2 * Hkv) * D, E, generator=g) / math.sqrt(E)).to(BF)
    inv = 10000.0 ** (-torch.arange(D // 2, dtype=torch.float64) * 2.0 / D)
    ang = torch.arange(S, dtype=torch.float64)[:, None] * inv[None, :]
    cos_t, sin_t = torch.cos(ang).float().contiguous(), torch.sin(ang).float().contiguous()
    q = hp.Guarded((B, H, S, D), BF)
    k, v = (hp.Guarded((B, Hkv, S, D), BF) for _ in range(2))
    mgn.mgn_qkv_rope_fwd(x.cuda(), w.cuda(), cos_t.cuda(), sin_t.cuda(), q.view, k.view, v.view, MODE)
    mgn.mgn_attn_check()
    rq, rk, rv = orc.qkv_rope(x.double().numpy(), w.double().numpy(), cos_t.double().numpy(), sin_t.double().numpy(), H, Hkv, D)
    for name, got, ref in (("Q", q, rq), ("K", k, rk), ("V", v, rv)):
        err = hp.rel_l2(got.check(name).double().numpy(), ref)
        assert err <= hp.FAST_REL_L2, f"{name}: {err:.3e}"


QKV_SHAPES = [
    # B, S, E, H, Hkv, D
    (1, 128, 64, 2, 2, 128),       # one tile
    (2, 197, 200, 3, 1, 64),       # ragged rows, E not a slice multiple, (H + 2 Hkv) D = 320: a row tile past the last head
    (1, 300, 512, 5, 5, 128),      # odd head count
    (3, 1, 8, 4, 2, 64),           # a single position
    (2, 520, 1024, 8, 2, 128),     # grouped key/value heads, several row tiles and contraction slices
]


def _qkv_case(seed, B, S, E, H, Hkv, D):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(B, S, E, generator=g).to(BF)
    w = (torch.randn((H + 2 * Hkv) * D, E, generator=g) / math.sqrt(E)).to(BF)
    inv = 10000.0 ** (-torch.arange(D // 2, dtype=torch.float64) * 2.0 / D)
    ang = torch.arange(S, dtype=torch.float64)[:, None] * inv[None, :]
    cos_t, sin_t = torch.cos(ang).float().contiguous(), torch.sin(ang).float().contiguous()
    g_q = torch.randn(B, H, S, D, generator=g).to(BF)
    g_k = torch.randn(B, Hkv, S, D, generator=g).to(BF)
    g_v = torch.randn(B, Hkv, S, D, generator=g).to(BF)
    return x, w, cos_t, sin_t, g_q, g_k, g_v


@pytest.mark.parametrize("B,S,E,H,Hkv,D", QKV_SHAPES)
def test_gradient_of_the_rotary_embedding_in_place(B, S, E, H, Hkv, D):
    x, w, cos_t, sin_t, g_q, g_k, g_v = _qkv_case(60 + S, B, S, E, H, Hkv, D)
    dq, dk = hp.Guarded((B, H, S, D), BF), hp.Guarded((B, Hkv, S, D), BF)
    dq.view.copy_(g_q); dk.view.copy_(g_k)
    mgn.mgn_rope_bwd_inplace(dq.view, dk.view, cos_t.cuda(), sin_t.cuda(), MODE)
    mgn.mgn_attn_check()
    _, _, gy = orc.qkv_rope_bwd(g_q.double().numpy(), g_k.double().numpy(), g_v.double().numpy(), x.double().numpy(),
                                w.double().numpy(), cos_t.double().numpy(), sin_t.double().numpy())
    ref_q = gy[..., : H * D].reshape(B, S, H, D).transpose(0, 2, 1, 3)
    ref_k = gy[..., H * D:(H + Hkv) * D].reshape(B, S, Hkv, D).transpose(0, 2, 1, 3)
    # one rounding to bf16 of an f32 result: relative 2^-9 per element
    assert hp.rel_l2(dq.check("dq").double().numpy(), ref_q) <= 3e-3
    assert hp.rel_l2(dk.check("dk").double().numpy(), ref_k) <= 3e-3


@pytest.mark.parametrize("B,S,E,H,Hkv,D", QKV_SHAPES)
def test_qkv_projection_backward_against_the_oracle(B, S, E, H, Hkv, D):
    """The three calls in sequence -- opposite rotation in place, data gradient, weight gradient -- against the
    oracle's backward of the rotated projection."""
    x, w, cos_t, sin_t, g_q, g_k, g_v = _qkv_case(70 + S, B, S, E, H, Hkv, D)
    dq, dk, dv = g_q.cuda(), g_k.cuda(), g_v.cuda()
    mgn.mgn_rope_bwd_inplace(dq, dk, cos_t.cuda(), sin_t.cuda(), MODE)
    dx = hp.Guarded((B, S, E), BF)
    dw = hp.Guarded(((H + 2 * Hkv) * D, E), BF)
    mgn.mgn_qkv_bwd_data(dq, dk, dv, w.cuda(), dx.view, MODE)
    mgn.mgn_qkv_bwd_weight(dq, dk, dv, x.cuda(), dw.view, MODE)
    mgn.mgn_attn_check()
    assert torch.equal(dv.cpu(), g_v)                       # the value gradient is only read
    rdx, rdw, _ = orc.qkv_rope_bwd(g_q.double().numpy(), g_k.double().numpy(), g_v.double().numpy(), x.double().numpy(),
                                   w.double().numpy(), cos_t.double().numpy(), sin_t.double().numpy())
    e_dx, e_dw = hp.rel_l2(dx.check("dX").double().numpy(), rdx), hp.rel_l2(dw.check("dW").double().numpy(), rdw)
    assert e_dx <= hp.FAST_REL_L2, f"dX: {e_dx:.3e}"
    assert e_dw <= hp.FAST_REL_L2, f"dW: {e_dw:.3e}"


def test_whole_layer_backward_chain():
    """dY -> output-projection backward (dO, delta) -> attention backward with that delta -> opposite rotation ->
    QKV data gradient, on tensors produced by this library's own forward chain; against the same chain in the
    oracle (f64 on the bf16-rounded inputs)."""
    B, S, E, H, Hkv, D = 1, 384, 256, 4, 2, 64
    x, w, cos_t, sin_t, _, _, _ = _qkv_case(91, B, S, E, H, Hkv, D)
    g = torch.Generator().manual_seed(92)
    w_o = (torch.randn(H * D, E, generator=g) / math.sqrt(H * D)).to(BF)
    d_y = torch.randn(B, S, E, generator=g).to(BF)
    scale = 1.0 / math.sqrt(D)
    xd, wd, wod, cd, sd = x.cuda(), w.cuda(), w_o.cuda(), cos_t.cuda(), sin_t.cuda()
    q = torch.empty(B, H, S, D, dtype=BF, device="cuda")
    k, v = (torch.empty(B, Hkv, S, D, dtype=BF, device="cuda") for _ in range(2))
    mgn.mgn_qkv_rope_fwd(xd, wd, cd, sd, q, k, v, MODE)
    o = torch.empty_like(q); lse = torch.empty(B, H, S, device="cuda")
    mgn.mgn_attn_fwd_ext(q, k, v, o, lse, True, scale, MODE)
    d_o = torch.empty_like(q); delta = torch.empty(B, H, S, device="cuda")
    mgn.mgn_out_proj_bwd_data(d_y.cuda(), wod, o, d_o, delta, MODE)
    dq = torch.empty_like(q); dk, dv = torch.empty_like(k), torch.empty_like(v)
    ws = mgn.alloc_workspace(B, H, S, D, MODE)
    mgn.mgn_attn_bwd_given_delta(q, k, v, d_o, lse, delta, dq, dk, dv, ws, True, scale, MODE)
    mgn.mgn_rope_bwd_inplace(dq, dk, cd, sd, MODE)
    dx = hp.Guarded((B, S, E), BF)
    mgn.mgn_qkv_bwd_data(dq, dk, dv, wd, dx.view, MODE)
    mgn.mgn_attn_check()
    # oracle chain
    c64, s64 = cos_t.double().numpy(), sin_t.double().numpy()
    rq, rk, rv = orc.qkv_rope(x.double().numpy(), w.double().numpy(), c64, s64, H, Hkv, D)
    r_do, _, _ = orc.out_proj_bwd(d_y.double().numpy(), w_o.double().numpy(), np.zeros((B, H, S, D)))
    ref = hp.run_oracle_ext(torch.from_numpy(rq), torch.from_numpy(rk), torch.from_numpy(rv), torch.from_numpy(r_do), True, scale)
    rdx, _, _ = orc.qkv_rope_bwd(ref["dQ"], ref["dK"], ref["dV"], x.double().numpy(), w.double().numpy(), c64, s64)
    err = hp.rel_l2(dx.check("dX").double().numpy(), rdx)
    assert err <= hp.FAST_REL_L2, f"dX through the whole layer: {err:.3e}"

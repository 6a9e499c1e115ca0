"""Pins of the extended-shape oracle (oracle/attn_ref_ext.c): separate query / key lengths and
grouped key/value heads.  None of them calls the function under test to make its own expectation:
they go through the square multi-head oracle (attn_ref.c, itself pinned in test_oracle_pins.py),
through a dense torch float64 evaluation with autograd, and through central finite differences.

Definition pinned (textbook; the paper's workload table names the cross-attention shapes but prints
no formula): query head h reads key/value head h // (H / H_kv); with a causal mask, key j is
visible to query i iff j <= i + (S_k - S_q)."""
import math

import numpy as np
import pytest
import torch

from oracle import attn_oracle as orc

RNG = np.random.default_rng(20260802)


def rand(*shape):
    return RNG.standard_normal(shape)


def test_reduces_to_the_square_multi_head_oracle():
    B, H, S, D = 2, 3, 37, 8
    q, k, v, d_o = rand(B, H, S, D), rand(B, H, S, D), rand(B, H, S, D), rand(B, H, S, D)
    for causal in (False, True):
        o0, l0, dq0, dk0, dv0 = orc.attn_bwd(q, k, v, d_o, causal, 0.3)
        o1, l1, dq1, dk1, dv1 = orc.attn_bwd_ext(q, k, v, d_o, causal, 0.3)
        of, lf = orc.attn_fwd_ext(q, k, v, causal, 0.3)
        for a, b in ((o0, o1), (l0, l1), (dq0, dq1), (dk0, dk1), (dv0, dv1), (o0, of), (l0, lf)):
            np.testing.assert_allclose(b, a, rtol=0, atol=1e-14)


@pytest.mark.parametrize("causal", [False, True])
def test_grouped_heads_equal_repeated_heads_with_summed_key_value_gradients(causal):
    B, H, Hkv, Sq, Sk, D = 2, 6, 2, 19, 19, 8
    G = H // Hkv
    q, d_o = rand(B, H, Sq, D), rand(B, H, Sq, D)
    k, v = rand(B, Hkv, Sk, D), rand(B, Hkv, Sk, D)
    k_rep, v_rep = np.repeat(k, G, axis=1), np.repeat(v, G, axis=1)     # head h reads h // G
    o0, l0, dq0, dk0, dv0 = orc.attn_bwd(q, k_rep, v_rep, d_o, causal, 0.4)
    o1, l1, dq1, dk1, dv1 = orc.attn_bwd_ext(q, k, v, d_o, causal, 0.4)
    np.testing.assert_allclose(o1, o0, atol=1e-14)
    np.testing.assert_allclose(l1, l0, atol=1e-14)
    np.testing.assert_allclose(dq1, dq0, atol=1e-13)
    np.testing.assert_allclose(dk1, dk0.reshape(B, Hkv, G, Sk, D).sum(axis=2), atol=1e-13)
    np.testing.assert_allclose(dv1, dv0.reshape(B, Hkv, G, Sk, D).sum(axis=2), atol=1e-13)


def test_bottom_right_causal_equals_the_last_rows_of_a_square_causal_problem():
    """Queries are the last S_q positions of an S_k-long sequence: pad Q with arbitrary earlier rows
    whose upstream gradient is zero; their rows of P do not touch the later rows, and with d_o = 0
    they add nothing to dK, dV."""
    B, H, Sq, Sk, D = 1, 2, 5, 13, 4
    q, d_o = rand(B, H, Sq, D), rand(B, H, Sq, D)
    k, v = rand(B, H, Sk, D), rand(B, H, Sk, D)
    q_pad = np.concatenate([rand(B, H, Sk - Sq, D), q], axis=2)
    do_pad = np.concatenate([np.zeros((B, H, Sk - Sq, D)), d_o], axis=2)
    o0, l0, dq0, dk0, dv0 = orc.attn_bwd(q_pad, k, v, do_pad, True, 0.5)
    o1, l1, dq1, dk1, dv1 = orc.attn_bwd_ext(q, k, v, d_o, True, 0.5)
    np.testing.assert_allclose(o1, o0[:, :, Sk - Sq:], atol=1e-14)
    np.testing.assert_allclose(l1, l0[:, :, Sk - Sq:], atol=1e-14)
    np.testing.assert_allclose(dq1, dq0[:, :, Sk - Sq:], atol=1e-13)
    np.testing.assert_allclose(dk1, dk0, atol=1e-13)
    np.testing.assert_allclose(dv1, dv0, atol=1e-13)


def _torch_dense(q, k, v, d_o, causal, scale):
    """Dense float64 evaluation with autograd: a third implementation."""
    tq, tk, tv = (torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (q, k, v))
    B, H, Sq, D = q.shape
    Hkv, Sk = k.shape[1], k.shape[2]
    G = H // Hkv
    idx = torch.arange(H) // G
    s = scale * torch.einsum("bhid,bhjd->bhij", tq, tk[:, idx])
    if causal:
        i = torch.arange(Sq)[:, None]
        j = torch.arange(Sk)[None, :]
        s = s.masked_fill(j > i + (Sk - Sq), float("-inf"))
    lse = torch.logsumexp(s, dim=-1)
    o = torch.einsum("bhij,bhjd->bhid", torch.softmax(s, dim=-1), tv[:, idx])
    o.backward(torch.tensor(d_o, dtype=torch.float64))
    return o.detach().numpy(), lse.detach().numpy(), tq.grad.numpy(), tk.grad.numpy(), tv.grad.numpy()


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal", [
    (1, 4, 4, 50, 16, 8, False),      # more queries than keys (action tokens over context tokens)
    (2, 8, 2, 33, 77, 16, False),     # text cross-attention length, grouped heads
    (1, 6, 3, 21, 40, 8, True),       # causal, bottom-right aligned, grouped
    (1, 2, 1, 1, 9, 4, True),         # a single query sees every key (decode-shaped row)
    (1, 3, 1, 7, 7, 4, True),         # multi-query attention, square causal
])
def test_against_torch_float64_autograd(B, H, Hkv, Sq, Sk, D, causal):
    q, d_o = rand(B, H, Sq, D), rand(B, H, Sq, D)
    k, v = rand(B, Hkv, Sk, D), rand(B, Hkv, Sk, D)
    scale = 1.0 / math.sqrt(D)
    ref = _torch_dense(q, k, v, d_o, causal, scale)
    got = orc.attn_bwd_ext(q, k, v, d_o, causal, scale)
    for a, b in zip(ref, got):
        np.testing.assert_allclose(b, a, rtol=1e-11, atol=1e-12)
    of, lf = orc.attn_fwd_ext(q, k, v, causal, scale)
    np.testing.assert_allclose(of, ref[0], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(lf, ref[1], rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("causal", [False, True])
def test_central_finite_differences(causal):
    B, H, Hkv, Sq, Sk, D = 1, 4, 2, 3, 5, 3
    q, d_o = rand(B, H, Sq, D), rand(B, H, Sq, D)
    k, v = rand(B, Hkv, Sk, D), rand(B, Hkv, Sk, D)
    scale = 0.7
    _, _, dq, dk, dv = orc.attn_bwd_ext(q, k, v, d_o, causal, scale)

    def loss(q_, k_, v_):
        o, _ = orc.attn_fwd_ext(q_, k_, v_, causal, scale)
        return float((o * d_o).sum())

    eps = 1e-6
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        flat = x.reshape(-1)
        for t in RNG.choice(flat.size, size=12, replace=False):
            old = flat[t]
            flat[t] = old + eps
            lp = loss(q, k, v)
            flat[t] = old - eps
            lm = loss(q, k, v)
            flat[t] = old
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - g.reshape(-1)[t]) <= 1e-7 * max(1.0, abs(fd)), (name, t, fd, g.reshape(-1)[t])


def test_softmax_rows_and_shape_errors():
    q, k, v = rand(1, 2, 4, 4), rand(1, 2, 9, 4), np.ones((1, 2, 9, 4))
    o, _ = orc.attn_fwd_ext(q, k, v, True, 1.0)
    np.testing.assert_allclose(o, 1.0, atol=1e-14)          # rows of P sum to one, also under the offset mask
    with pytest.raises(ValueError):
        orc.attn_fwd_ext(rand(1, 2, 9, 4), rand(1, 2, 4, 4), rand(1, 2, 4, 4), True, 1.0)   # causal, S_q > S_k
    with pytest.raises(AssertionError):
        orc.attn_fwd_ext(rand(1, 3, 4, 4), rand(1, 2, 4, 4), rand(1, 2, 4, 4), False, 1.0)  # H % H_kv != 0


def test_hand_worked_grouped_head_example():
    """tests/golden/hand_case_grouped_heads.json: exact fractions derived by hand (see its citation)."""
    import json
    import os
    fx = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_case_grouped_heads.json")))
    q = np.array(fx["Q"]).reshape(1, 2, 1, 1)
    k = np.array(fx["K"]).reshape(1, 1, 2, 1)
    v = np.array(fx["V"]).reshape(1, 1, 2, 1)
    d_o = np.array(fx["dO"]).reshape(1, 2, 1, 1)
    assert abs(fx["ln2"] - math.log(2)) < 1e-15 and abs(fx["ln3"] - math.log(3)) < 1e-15
    o, lse, dq, dk, dv = orc.attn_bwd_ext(q, k, v, d_o, False, fx["scale"])
    np.testing.assert_allclose(o.reshape(2), np.array(fx["O"]).reshape(2), atol=1e-14)
    np.testing.assert_allclose(lse.reshape(2), np.array(fx["LSE"]), atol=1e-14)
    np.testing.assert_allclose(dq.reshape(2), np.array(fx["dQ"]).reshape(2), atol=1e-14)
    np.testing.assert_allclose(dk.reshape(2), np.array(fx["dK"]).reshape(2), atol=1e-14)
    np.testing.assert_allclose(dv.reshape(2), np.array(fx["dV"]).reshape(2), atol=1e-14)
    # the causal mask of a single query over two keys is bottom-right aligned: the query sees both keys
    oc, lsec, dqc, dkc, dvc = orc.attn_bwd_ext(q, k, v, d_o, True, fx["scale"])
    for a, b in ((o, oc), (lse, lsec), (dq, dqc), (dk, dkc), (dv, dvc)):
        np.testing.assert_allclose(b, a, atol=1e-15)

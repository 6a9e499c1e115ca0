"""Pins for the CPU oracle: everything here fixes oracle/attn_ref.c against the
mathematics, a hand-worked example, a separately written dense evaluation and a
third implementation (torch float64 CPU attention with autograd).  No GPU."""
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import attn_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rnd(seed, *shape):
    return np.random.default_rng(seed).standard_normal(shape)


def one_head(x):
    return x[None, None]


# --------------------------------------------------------------------------- worked example
@pytest.mark.parametrize("mask", ["noncausal", "causal"])
def test_hand_worked_example(mask):
    g = json.load(open(os.path.join(GOLDEN, "hand_case_s2_d2.json")))
    Q, K, V, dO = (np.array(g[n], dtype=np.float64) for n in ("Q", "K", "V", "dO"))
    exp = g[mask]
    causal = mask == "causal"
    o, lse = orc.attn_fwd(one_head(Q), one_head(K), one_head(V), causal, g["scale"])
    o2, lse2, dq, dk, dv = orc.attn_bwd(one_head(Q), one_head(K), one_head(V), one_head(dO),
                                        causal, g["scale"])
    P, dP, dS = orc.head_matrices(Q, K, V, dO, causal, g["scale"])
    tol = dict(rtol=0, atol=1e-14)
    np.testing.assert_allclose(o[0, 0], exp["O"], **tol)
    np.testing.assert_allclose(o2[0, 0], exp["O"], **tol)
    np.testing.assert_allclose(lse[0, 0], exp["LSE"], **tol)
    np.testing.assert_allclose(lse2[0, 0], exp["LSE"], **tol)
    np.testing.assert_allclose(P, exp["P"], **tol)
    np.testing.assert_allclose(dS, exp["dS"], **tol)
    np.testing.assert_allclose(dq[0, 0], exp["dQ"], **tol)
    np.testing.assert_allclose(dk[0, 0], exp["dK"], **tol)
    np.testing.assert_allclose(dv[0, 0], exp["dV"], **tol)


# --------------------------------------------------------------------------- dense evaluation
def dense_eval(Q, K, V, dO, causal, scale):
    """Literal matrix form, one head, numpy: written independently of the C oracle."""
    S = Q.shape[0]
    s = scale * (Q @ K.T)
    if causal:
        s = np.where(np.tril(np.ones((S, S), dtype=bool)), s, -np.inf)
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    l = e.sum(axis=1, keepdims=True)
    P = e / l
    lse = (m + np.log(l))[:, 0]
    O = P @ V
    dV = P.T @ dO
    dP = dO @ V.T
    delta = (dO * O).sum(axis=1, keepdims=True)
    dS = P * (dP - delta)
    dQ = scale * dS @ K
    dK = scale * dS.T @ Q
    return dict(O=O, LSE=lse, P=P, dS=dS, dQ=dQ, dK=dK, dV=dV)


@pytest.mark.parametrize("S,D", [(1, 4), (2, 3), (5, 2), (16, 8), (33, 16), (70, 32)])
@pytest.mark.parametrize("causal", [False, True])
def test_matches_dense_matrix_form(S, D, causal):
    Q, K, V, dO = (rnd(100 + t + S, S, D) for t in range(4))
    scale = 0.37
    ref = dense_eval(Q, K, V, dO, causal, scale)
    o, lse = orc.attn_fwd(one_head(Q), one_head(K), one_head(V), causal, scale)
    o2, lse2, dq, dk, dv = orc.attn_bwd(*(one_head(x) for x in (Q, K, V, dO)), causal, scale)
    P, dP, dS = orc.head_matrices(Q, K, V, dO, causal, scale)
    tol = dict(rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(o[0, 0], ref["O"], **tol)
    np.testing.assert_allclose(o2[0, 0], o[0, 0], rtol=0, atol=0)
    np.testing.assert_allclose(lse2[0, 0], lse[0, 0], rtol=0, atol=0)
    np.testing.assert_allclose(lse[0, 0], ref["LSE"], **tol)
    np.testing.assert_allclose(P, ref["P"], **tol)
    visible = np.tril(np.ones((S, S), dtype=bool)) if causal else np.ones((S, S), dtype=bool)
    np.testing.assert_allclose(dP, np.where(visible, dO @ V.T, 0.0), **tol)   # dP on its own (masked entries are 0)
    np.testing.assert_allclose(dS, ref["dS"], **tol)
    np.testing.assert_allclose(dq[0, 0], ref["dQ"], **tol)
    np.testing.assert_allclose(dk[0, 0], ref["dK"], **tol)
    np.testing.assert_allclose(dv[0, 0], ref["dV"], **tol)


# --------------------------------------------------------------------------- third implementation
@pytest.mark.parametrize("B,H,S,D", [(2, 3, 17, 8), (1, 2, 64, 32)])
@pytest.mark.parametrize("causal", [False, True])
def test_matches_torch_float64_autograd(B, H, S, D, causal):
    g = torch.Generator().manual_seed(7 + S)
    q, k, v, d_o = (torch.randn(B, H, S, D, generator=g, dtype=torch.float64) for _ in range(4))
    scale = 1.0 / math.sqrt(D)
    qt, kt, vt = (x.clone().requires_grad_(True) for x in (q, k, v))
    out = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=causal, scale=scale)
    out.backward(d_o)
    s = scale * q @ k.transpose(-1, -2)
    if causal:
        s = s.masked_fill(~torch.tril(torch.ones(S, S, dtype=torch.bool)), float("-inf"))
    lse_t = torch.logsumexp(s, dim=-1)
    o, lse, dq, dk, dv = orc.attn_bwd(q.numpy(), k.numpy(), v.numpy(), d_o.numpy(), causal, scale)
    tol = dict(rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(o, out.detach().numpy(), **tol)
    np.testing.assert_allclose(lse, lse_t.numpy(), **tol)
    np.testing.assert_allclose(dq, qt.grad.numpy(), **tol)
    np.testing.assert_allclose(dk, kt.grad.numpy(), **tol)
    np.testing.assert_allclose(dv, vt.grad.numpy(), **tol)


# --------------------------------------------------------------------------- finite differences
@pytest.mark.parametrize("S,D", [(4, 2), (7, 8), (16, 4)])
@pytest.mark.parametrize("causal", [False, True])
def test_gradients_by_central_finite_differences(S, D, causal):
    B, H = 1, 2
    q, k, v, d_o = (rnd(200 + t + S, B, H, S, D) for t in range(4))
    scale = 0.6
    _, _, dq, dk, dv = orc.attn_bwd(q, k, v, d_o, causal, scale)

    def loss(q_, k_, v_):
        o, _ = orc.attn_fwd(q_, k_, v_, causal, scale)
        return float((o * d_o).sum())

    h = 1e-6
    rng = np.random.default_rng(5)
    for name, x, grad in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        fd = np.zeros_like(x)
        idx = [tuple(rng.integers(0, n) for n in x.shape) for _ in range(24)]
        idx += [(0, 0, 0, 0), (0, H - 1, S - 1, D - 1)]
        for ix in idx:
            xp, xm = x.copy(), x.copy()
            xp[ix] += h
            xm[ix] -= h
            args_p = dict(q=q, k=k, v=v); args_p[name] = xp
            args_m = dict(q=q, k=k, v=v); args_m[name] = xm
            fd_val = (loss(args_p["q"], args_p["k"], args_p["v"]) -
                      loss(args_m["q"], args_m["k"], args_m["v"])) / (2 * h)
            assert abs(fd_val - grad[ix]) <= 1e-7 * max(1.0, abs(grad[ix])), (name, ix, fd_val, grad[ix])


# --------------------------------------------------------------------------- row identities
@pytest.mark.parametrize("causal", [False, True])
def test_row_identities(causal):
    S, D = 40, 16
    Q, K, V, dO = (rnd(300 + t, S, D) for t in range(4))
    scale = 0.25
    P, dP, dS = orc.head_matrices(Q, K, V, dO, causal, scale)
    assert np.abs(P.sum(axis=1) - 1).max() <= 1e-14
    assert (P >= 0).all()
    if causal:
        assert np.abs(np.triu(P, 1)).max() == 0.0
        assert np.abs(np.triu(dS, 1)).max() == 0.0
    assert np.abs(dS.sum(axis=1)).max() <= 1e-13
    o, _ = orc.attn_fwd(one_head(Q), one_head(K), one_head(V), causal, scale)
    delta_a = (dO * o[0, 0]).sum(axis=1)
    delta_b = (P * dP).sum(axis=1)
    np.testing.assert_allclose(delta_a, delta_b, rtol=0, atol=1e-13)


# --------------------------------------------------------------------------- closed forms
@pytest.mark.parametrize("causal", [False, True])
def test_identical_keys_closed_form(causal):
    S, D = 12, 6
    Q, V, dO = rnd(1, S, D), rnd(2, S, D), rnd(3, S, D)
    kvec = rnd(4, D)
    K = np.tile(kvec, (S, 1))
    scale = 0.7
    o, lse, dq, dk, dv = orc.attn_bwd(*(one_head(x) for x in (Q, K, V, dO)), causal, scale)
    n = np.arange(1, S + 1) if causal else np.full(S, S)
    mean_v = np.cumsum(V, axis=0) / n[:, None] if causal else np.tile(V.mean(axis=0), (S, 1))
    np.testing.assert_allclose(o[0, 0], mean_v, rtol=0, atol=1e-14)
    np.testing.assert_allclose(lse[0, 0], scale * Q @ kvec + np.log(n), rtol=0, atol=1e-14)
    # sum_j dS_ij = 0 and all key rows equal  =>  dQ = 0
    assert np.abs(dq).max() <= 1e-14
    # dV_j = sum_i P_ij dO_i with uniform P
    if causal:
        w = np.where(np.tril(np.ones((S, S), dtype=bool)), 1.0 / n[:, None], 0.0)
    else:
        w = np.full((S, S), 1.0 / S)
    np.testing.assert_allclose(dv[0, 0], w.T @ dO, rtol=0, atol=1e-14)


def test_single_key():
    D = 5
    Q, K, V, dO = rnd(1, 1, D), rnd(2, 1, D), rnd(3, 1, D), rnd(4, 1, D)
    for causal in (False, True):
        o, lse, dq, dk, dv = orc.attn_bwd(*(one_head(x) for x in (Q, K, V, dO)), causal, 1.3)
        np.testing.assert_allclose(o[0, 0], V, rtol=0, atol=0)
        np.testing.assert_allclose(lse[0, 0], 1.3 * (Q @ K.T)[0], rtol=0, atol=1e-15)
        np.testing.assert_allclose(dv[0, 0], dO, rtol=0, atol=0)
        assert np.abs(dq).max() == 0 and np.abs(dk).max() == 0


@pytest.mark.parametrize("causal", [False, True])
def test_zero_ds_cases(causal):
    S, D = 9, 4
    Q, K, dO = rnd(1, S, D), rnd(2, S, D), rnd(3, S, D)
    # (ii) all V rows identical => O_i = v and dS = 0 for any Q, K, dO
    vvec = rnd(4, D)
    V = np.tile(vvec, (S, 1))
    o, lse, dq, dk, dv = orc.attn_bwd(*(one_head(x) for x in (Q, K, V, dO)), causal, 0.5)
    np.testing.assert_allclose(o[0, 0], V, rtol=0, atol=1e-14)
    assert np.abs(dq).max() <= 1e-14 and np.abs(dk).max() <= 1e-14
    # (i) dO constant within each row and every V row with the same row-sum => dS = 0
    V2 = rnd(5, S, D)
    V2[:, -1] += 2.0 - V2.sum(axis=1)
    dO2 = np.tile(rnd(6, S, 1), (1, D))
    _, _, dS = orc.head_matrices(Q, K, V2, dO2, causal, 0.5)
    assert np.abs(dS).max() <= 1e-14
    # and the counter-example: generic V gives a non-zero dS for the same dO
    _, _, dS3 = orc.head_matrices(Q, K, rnd(7, S, D), dO2, causal, 0.5)
    assert np.abs(dS3).max() > 1e-3


def test_scale_zero_is_uniform_attention():
    S, D = 6, 3
    Q, K, V = rnd(1, S, D), rnd(2, S, D), rnd(3, S, D)
    o, lse = orc.attn_fwd(one_head(Q), one_head(K), one_head(V), False, 0.0)
    np.testing.assert_allclose(o[0, 0], np.tile(V.mean(axis=0), (S, 1)), rtol=0, atol=1e-15)
    np.testing.assert_allclose(lse[0, 0], np.full(S, math.log(S)), rtol=0, atol=1e-15)


# --------------------------------------------------------------------------- invariances
def test_key_shift_and_permutation_invariance():
    S, D = 14, 5
    Q, K, V = rnd(1, S, D), rnd(2, S, D), rnd(3, S, D)
    scale = 0.4
    c = rnd(4, D)
    for causal in (False, True):
        o, lse = orc.attn_fwd(one_head(Q), one_head(K), one_head(V), causal, scale)
        o2, lse2 = orc.attn_fwd(one_head(Q), one_head(K + c), one_head(V), causal, scale)
        np.testing.assert_allclose(o2, o, rtol=0, atol=1e-13)
        np.testing.assert_allclose(lse2[0, 0], lse[0, 0] + scale * Q @ c, rtol=0, atol=1e-13)
    perm = np.random.default_rng(9).permutation(S)
    o, lse = orc.attn_fwd(one_head(Q), one_head(K), one_head(V), False, scale)
    o3, lse3 = orc.attn_fwd(one_head(Q), one_head(K[perm]), one_head(V[perm]), False, scale)
    np.testing.assert_allclose(o3, o, rtol=0, atol=1e-14)
    np.testing.assert_allclose(lse3, lse, rtol=0, atol=1e-14)


def test_ds_products_swap_identity():
    S, D = 11, 7
    dS, Q, K = rnd(1, S, S), rnd(2, S, D), rnd(3, S, D)
    dq, dk = orc.grads_from_ds(dS, Q, K, 0.3)
    dq_sw, dk_sw = orc.grads_from_ds(dS.T.copy(), K, Q, 0.3)
    np.testing.assert_allclose(dq_sw, dk, rtol=0, atol=1e-14)
    np.testing.assert_allclose(dk_sw, dq, rtol=0, atol=1e-14)
    np.testing.assert_allclose(dq, 0.3 * dS @ K, rtol=0, atol=1e-13)
    # the full backward uses the same two products of its own dS
    V, dO = rnd(4, S, D), rnd(5, S, D)
    _, _, dS_full = orc.head_matrices(Q, K, V, dO, False, 0.3)
    _, _, dq_b, dk_b, _ = orc.attn_bwd(*(one_head(x) for x in (Q, K, V, dO)), False, 0.3)
    dq_p, dk_p = orc.grads_from_ds(dS_full, Q, K, 0.3)
    np.testing.assert_allclose(dq_b[0, 0], dq_p, rtol=0, atol=1e-14)
    np.testing.assert_allclose(dk_b[0, 0], dk_p, rtol=0, atol=1e-14)


@pytest.mark.parametrize("causal", [False, True])
def test_inner_product_invariants(causal):
    B, H, S, D = 2, 2, 37, 16
    q, k, v, d_o = (rnd(400 + t, B, H, S, D) for t in range(4))
    o, lse, dq, dk, dv = orc.attn_bwd(q, k, v, d_o, causal, 0.25)
    for b in range(B):
        for h in range(H):
            i1a, i1b = (dq[b, h] * q[b, h]).sum(), (dk[b, h] * k[b, h]).sum()
            i2a, i2b = (dv[b, h] * v[b, h]).sum(), (d_o[b, h] * o[b, h]).sum()
            assert abs(i1a - i1b) <= 1e-12 * max(1, abs(i1a))
            assert abs(i2a - i2b) <= 1e-12 * max(1, abs(i2a))


def test_heads_are_independent_and_laid_out_bhsd():
    B, H, S, D = 2, 3, 10, 4
    q, k, v, d_o = (rnd(500 + t, B, H, S, D) for t in range(4))
    o, lse, dq, dk, dv = orc.attn_bwd(q, k, v, d_o, True, 0.5, nthreads=3)
    of, lsef = orc.attn_fwd(q, k, v, True, 0.5, nthreads=2)
    np.testing.assert_array_equal(of, o)
    np.testing.assert_array_equal(lsef, lse)
    for b in range(B):
        for h in range(H):
            o1, l1, dq1, dk1, dv1 = orc.attn_bwd(*(x[b:b + 1, h:h + 1] for x in (q, k, v, d_o)), True, 0.5)
            np.testing.assert_array_equal(o1[0, 0], o[b, h])
            np.testing.assert_array_equal(l1[0, 0], lse[b, h])
            np.testing.assert_array_equal(dq1[0, 0], dq[b, h])
            np.testing.assert_array_equal(dk1[0, 0], dk[b, h])
            np.testing.assert_array_equal(dv1[0, 0], dv[b, h])

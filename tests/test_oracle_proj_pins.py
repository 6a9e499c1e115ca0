"""Pins for the output-projection oracle (oracle/proj_ref.c): none of them goes through the function
under test.  A hand-worked example, central finite differences, torch float64 einsum + autograd,
the identity weight, linearity, and the delta identity of the attention backward.  No GPU."""
import numpy as np
import pytest
import torch

from oracle import attn_oracle as orc


def rnd(seed, *shape):
    return np.random.default_rng(seed).standard_normal(shape)


def test_hand_worked_example():
    # B=1, H=2, S=1, D=1, E=2: O = [3 | 5] (one row, two heads), W = [[1, 2], [-1, 4]]
    o = np.array([3.0, 5.0]).reshape(1, 2, 1, 1)
    w = np.array([[1.0, 2.0], [-1.0, 4.0]])
    y = orc.out_proj_fwd(o, w)
    np.testing.assert_allclose(y, np.array([[[3 - 5, 6 + 20]]], dtype=float), rtol=0, atol=0)   # [-2, 26]
    d_y = np.array([[[0.5, -1.0]]])
    d_o, delta, d_w = orc.out_proj_bwd(d_y, w, o)
    # dO_h = dY . W[h,:]: head 0: 0.5 - 2 = -1.5; head 1: -0.5 - 4 = -4.5
    np.testing.assert_allclose(d_o.ravel(), [-1.5, -4.5], rtol=0, atol=0)
    np.testing.assert_allclose(delta.ravel(), [-4.5, -22.5], rtol=0, atol=0)       # dO * O per head
    np.testing.assert_allclose(d_w, [[1.5, -3.0], [2.5, -5.0]], rtol=0, atol=0)    # O_h * dY


@pytest.mark.parametrize("B,H,S,D,E", [(2, 3, 5, 4, 7), (1, 2, 9, 8, 16)])
def test_matches_torch_float64_autograd(B, H, S, D, E):
    g = torch.Generator().manual_seed(B + S + E)
    o = torch.randn(B, H, S, D, generator=g, dtype=torch.float64, requires_grad=True)
    w = torch.randn(H * D, E, generator=g, dtype=torch.float64, requires_grad=True)
    d_y = torch.randn(B, S, E, generator=g, dtype=torch.float64)
    y = torch.einsum("bhsd,hde->bse", o, w.view(H, D, E))
    y.backward(d_y)
    tol = dict(rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(orc.out_proj_fwd(o.detach().numpy(), w.detach().numpy()), y.detach().numpy(), **tol)
    d_o, delta, d_w = orc.out_proj_bwd(d_y.numpy(), w.detach().numpy(), o.detach().numpy())
    np.testing.assert_allclose(d_o, o.grad.numpy(), **tol)
    np.testing.assert_allclose(d_w, w.grad.numpy(), **tol)
    np.testing.assert_allclose(delta, (o.grad * o.detach()).sum(-1).numpy(), **tol)


def test_central_finite_differences():
    B, H, S, D, E = 1, 2, 3, 2, 3
    o, w, d_y = rnd(1, B, H, S, D), rnd(2, H * D, E), rnd(3, B, S, E)
    loss = lambda o_, w_: float((orc.out_proj_fwd(o_, w_) * d_y).sum())
    d_o, _, d_w = orc.out_proj_bwd(d_y, w, o)
    h = 1e-6
    for idx in np.ndindex(o.shape):
        p, m = o.copy(), o.copy()
        p[idx] += h; m[idx] -= h
        assert abs((loss(p, w) - loss(m, w)) / (2 * h) - d_o[idx]) <= 1e-7
    for idx in np.ndindex(w.shape):
        p, m = w.copy(), w.copy()
        p[idx] += h; m[idx] -= h
        assert abs((loss(o, p) - loss(o, m)) / (2 * h) - d_w[idx]) <= 1e-7


def test_identity_weight_concatenates_heads_and_transposed_weight_swaps_roles():
    B, H, S, D = 2, 3, 4, 5
    o = rnd(4, B, H, S, D)
    y = orc.out_proj_fwd(o, np.eye(H * D))
    np.testing.assert_array_equal(y, o.transpose(0, 2, 1, 3).reshape(B, S, H * D))   # a dropped or swapped head fails
    d_y = rnd(5, B, S, H * D)
    d_o, delta, d_w = orc.out_proj_bwd(d_y, np.eye(H * D), o)
    np.testing.assert_array_equal(d_o, d_y.reshape(B, S, H, D).transpose(0, 2, 1, 3))
    np.testing.assert_allclose(delta, (d_o * o).sum(-1), rtol=1e-14, atol=1e-14)


def test_linearity_in_both_arguments():
    B, H, S, D, E = 1, 2, 6, 4, 5
    o1, o2, w1, w2 = rnd(6, B, H, S, D), rnd(7, B, H, S, D), rnd(8, H * D, E), rnd(9, H * D, E)
    f = orc.out_proj_fwd
    np.testing.assert_allclose(f(2 * o1 - o2, w1), 2 * f(o1, w1) - f(o2, w1), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(f(o1, w1 + 3 * w2), f(o1, w1) + 3 * f(o1, w2), rtol=1e-12, atol=1e-12)


def test_delta_is_the_row_statistic_of_the_attention_backward():
    """delta from the dO producer equals sum_j P_ij dP_ij of the attention oracle (delta two ways)."""
    S, D, E = 12, 4, 6
    q, k, v = rnd(10, S, D), rnd(11, S, D), rnd(12, S, D)
    w, d_y = rnd(13, D, E), rnd(14, 1, S, E)
    o, _ = orc.attn_fwd(q[None, None], k[None, None], v[None, None], True, 0.5)
    d_o, delta, _ = orc.out_proj_bwd(d_y, w, o)
    P, dP, _ = orc.head_matrices(q, k, v, d_o[0, 0], True, 0.5)
    np.testing.assert_allclose(delta[0, 0], (P * dP).sum(axis=1), rtol=1e-12, atol=1e-13)

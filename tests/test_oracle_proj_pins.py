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


# --------------------------------------------------------------------------- QKV projection + rotary embedding
def _angles(S, D, base=10000.0):
    inv = base ** (-np.arange(D // 2) * 2.0 / D)
    ang = np.arange(S)[:, None] * inv[None, :]
    return np.cos(ang), np.sin(ang)


def test_qkv_rope_hand_worked_example():
    # B=1, S=2, E=1, H=1, Hkv=1, D=2: y = x * w; position 0 is not rotated, position 1 by angle a
    x = np.array([[[2.0], [3.0]]])
    w = np.array([[1.0], [2.0], [-1.0], [0.5], [4.0], [5.0]])          # q: (1,2)  k: (-1,0.5)  v: (4,5)
    a = 0.3
    cos_t, sin_t = np.array([[1.0], [math_cos := np.cos(a)]]), np.array([[0.0], [math_sin := np.sin(a)]])
    q, k, v = orc.qkv_rope(x, w, cos_t, sin_t, 1, 1, 2)
    np.testing.assert_allclose(q[0, 0, 0], [2.0, 4.0], atol=1e-15)                    # x=2, no rotation
    np.testing.assert_allclose(q[0, 0, 1], [3 * math_cos - 6 * math_sin, 6 * math_cos + 3 * math_sin], atol=1e-15)
    np.testing.assert_allclose(k[0, 0, 1], [-3 * math_cos - 1.5 * math_sin, 1.5 * math_cos - 3 * math_sin], atol=1e-15)
    np.testing.assert_allclose(v[0, 0], [[8.0, 10.0], [12.0, 15.0]], atol=1e-15)      # values are not rotated


@pytest.mark.parametrize("B,S,E,H,Hkv,D", [(2, 5, 7, 3, 1, 4), (1, 9, 6, 2, 2, 8)])
def test_qkv_rope_matches_torch_float64(B, S, E, H, Hkv, D):
    g = torch.Generator().manual_seed(S + E)
    x = torch.randn(B, S, E, generator=g, dtype=torch.float64)
    w = torch.randn((H + 2 * Hkv) * D, E, generator=g, dtype=torch.float64)
    cos_t, sin_t = _angles(S, D)
    y = (x @ w.t()).view(B, S, H + 2 * Hkv, D).permute(0, 2, 1, 3)                     # [B, heads, S, D]
    c = torch.from_numpy(np.concatenate([cos_t, cos_t], axis=1))                        # rotate-half, written the usual way
    s_ = torch.from_numpy(np.concatenate([sin_t, sin_t], axis=1))
    rot = torch.cat([-y[..., D // 2:], y[..., :D // 2]], dim=-1)
    yr = y * c + rot * s_
    q, k, v = orc.qkv_rope(x.numpy(), w.numpy(), cos_t, sin_t, H, Hkv, D)
    tol = dict(rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(q, yr[:, :H].numpy(), **tol)
    np.testing.assert_allclose(k, yr[:, H:H + Hkv].numpy(), **tol)
    np.testing.assert_allclose(v, y[:, H + Hkv:].numpy(), **tol)


def test_qkv_rope_invariants():
    """A rotation keeps the norm of every (d, d + D/2) pair; q.k of rotated vectors depends only on the
    position difference; zero angles leave the plain projection."""
    B, S, E, H, Hkv, D = 1, 6, 5, 1, 1, 4
    x, w = rnd(20, B, S, E), rnd(21, (H + 2 * Hkv) * D, E)
    cos_t, sin_t = _angles(S, D)
    q, k, v = orc.qkv_rope(x, w, cos_t, sin_t, H, Hkv, D)
    q0, k0, v0 = orc.qkv_rope(x, w, np.ones_like(cos_t), np.zeros_like(sin_t), H, Hkv, D)
    np.testing.assert_allclose(v, v0, rtol=0, atol=0)
    np.testing.assert_allclose(q0[0, 0], x[0] @ w[:D].T, rtol=1e-13, atol=1e-13)
    pair_norm = lambda t: t[..., :D // 2] ** 2 + t[..., D // 2:] ** 2
    np.testing.assert_allclose(pair_norm(q), pair_norm(q0), rtol=1e-12, atol=1e-12)
    # the same unrotated vectors placed at positions (1, 3) and (2, 4) give the same rotated dot product
    xs = np.zeros((1, 6, E)); xs[0, 1] = xs[0, 2] = x[0, 0]; xs[0, 3] = xs[0, 4] = x[0, 5]
    q, k, _ = orc.qkv_rope(xs, w, cos_t, sin_t, H, Hkv, D)
    np.testing.assert_allclose(q[0, 0, 3] @ k[0, 0, 1], q[0, 0, 4] @ k[0, 0, 2], rtol=1e-12, atol=1e-12)


# ---- backward of the query/key/value projection with rotation --------------------------------------

def _angles_seeded(S, D, seed):
    th = np.random.default_rng(seed).uniform(-3.0, 3.0, (S, D // 2))
    return np.cos(th), np.sin(th)


def test_qkv_bwd_hand_worked_example():
    # B=1, S=1, E=1, H=1, Hkv=1, D=2, x = 2, w = [1, 3 | -1, 2 | 4, 5] (query | key | value rows),
    # angle with cos = 0, sin = 1: out[0] = -y[1], out[1] = y[0].
    x = np.array([[[2.0]]]); w = np.array([[1.0], [3.0], [-1.0], [2.0], [4.0], [5.0]])
    c, s = np.array([[0.0]]), np.array([[1.0]])
    q, k, v = orc.qkv_rope(x, w, c, s, 1, 1, 2)
    np.testing.assert_allclose(q.ravel(), [-6.0, 2.0]); np.testing.assert_allclose(k.ravel(), [-4.0, -2.0])
    g_q = np.array([1.0, 10.0]).reshape(1, 1, 1, 2); g_k = np.array([100.0, 1000.0]).reshape(1, 1, 1, 2)
    g_v = np.array([0.5, 0.25]).reshape(1, 1, 1, 2)
    dx, dw, gy = orc.qkv_rope_bwd(g_q, g_k, g_v, x, w, c, s)
    # q0 = -y1, q1 = y0  =>  gy0 = g_q1, gy1 = -g_q0
    np.testing.assert_allclose(gy.ravel(), [10.0, -1.0, 1000.0, -100.0, 0.5, 0.25], rtol=0, atol=0)
    np.testing.assert_allclose(dw.ravel(), 2.0 * gy.ravel(), rtol=0, atol=0)
    np.testing.assert_allclose(dx.ravel(), [10 - 3 - 1000 - 200 + 2 + 1.25], rtol=0, atol=1e-12)


@pytest.mark.parametrize("B,S,E,H,Hkv,D", [(2, 5, 7, 3, 1, 4), (1, 6, 5, 2, 2, 8)])
def test_qkv_bwd_matches_torch_float64_autograd(B, S, E, H, Hkv, D):
    g = torch.Generator().manual_seed(B + S + E + D)
    x = torch.randn(B, S, E, generator=g, dtype=torch.float64, requires_grad=True)
    w = torch.randn((H + 2 * Hkv) * D, E, generator=g, dtype=torch.float64, requires_grad=True)
    c, s = _angles_seeded(S, D, 5)
    ct, st = torch.from_numpy(c), torch.from_numpy(s)
    y = torch.einsum("bse,fe->bsf", x, w).view(B, S, H + 2 * Hkv, D).permute(0, 2, 1, 3)     # [B, heads, S, D]
    lo, hi = y[..., : D // 2], y[..., D // 2:]
    rot = torch.cat([lo * ct - hi * st, hi * ct + lo * st], dim=-1)
    q, k, v = rot[:, :H], rot[:, H:H + Hkv], y[:, H + Hkv:]
    g_q = torch.randn(q.shape, generator=g, dtype=torch.float64)
    g_k = torch.randn(k.shape, generator=g, dtype=torch.float64)
    g_v = torch.randn(v.shape, generator=g, dtype=torch.float64)
    ((q * g_q).sum() + (k * g_k).sum() + (v * g_v).sum()).backward()
    dx, dw, _ = orc.qkv_rope_bwd(g_q.numpy(), g_k.numpy(), g_v.numpy(), x.detach().numpy(), w.detach().numpy(), c, s)
    np.testing.assert_allclose(dx, x.grad.numpy(), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dw, w.grad.numpy(), rtol=1e-12, atol=1e-12)


def test_qkv_bwd_central_finite_differences_of_the_forward_oracle():
    B, S, E, H, Hkv, D = 1, 3, 3, 2, 1, 4
    x, w = rnd(11, B, S, E), rnd(12, (H + 2 * Hkv) * D, E)
    c, s = _angles_seeded(S, D, 13)
    g_q, g_k, g_v = rnd(14, B, H, S, D), rnd(15, B, Hkv, S, D), rnd(16, B, Hkv, S, D)

    def loss(x_, w_):
        q, k, v = orc.qkv_rope(x_, w_, c, s, H, Hkv, D)
        return float((q * g_q).sum() + (k * g_k).sum() + (v * g_v).sum())

    dx, dw, _ = orc.qkv_rope_bwd(g_q, g_k, g_v, x, w, c, s)
    h = 1e-6
    for idx in np.ndindex(x.shape):
        p, m = x.copy(), x.copy()
        p[idx] += h; m[idx] -= h
        assert abs((loss(p, w) - loss(m, w)) / (2 * h) - dx[idx]) <= 1e-6
    for idx in np.ndindex(w.shape):
        p, m = w.copy(), w.copy()
        p[idx] += h; m[idx] -= h
        assert abs((loss(x, p) - loss(x, m)) / (2 * h) - dw[idx]) <= 1e-6


def test_qkv_bwd_inverse_rotation_properties():
    """The gradient with respect to the unrotated projection is the rotation by the opposite angle: it keeps
    pair norms, undoes the forward rotation, and with zero angles it is the concatenation of the inputs."""
    B, S, E, H, Hkv, D = 2, 4, 3, 2, 1, 6
    x, w = rnd(21, B, S, E), rnd(22, (H + 2 * Hkv) * D, E)
    c, s = _angles_seeded(S, D, 23)
    q, k, v = orc.qkv_rope(x, w, c, s, H, Hkv, D)
    _, _, gy = orc.qkv_rope_bwd(q, k, v, x, w, c, s)              # feed the rotated outputs back
    y = np.einsum("bse,fe->bsf", x, w)                             # the unrotated projection
    np.testing.assert_allclose(gy, y, rtol=1e-12, atol=1e-12)      # R^T R = I
    g_q, g_k, g_v = rnd(24, B, H, S, D), rnd(25, B, Hkv, S, D), rnd(26, B, Hkv, S, D)
    _, _, gy2 = orc.qkv_rope_bwd(g_q, g_k, g_v, x, w, c, s)
    gq_un = gy2[..., : H * D].reshape(B, S, H, D).transpose(0, 2, 1, 3)
    half = D // 2
    np.testing.assert_allclose(gq_un[..., :half] ** 2 + gq_un[..., half:] ** 2,
                               g_q[..., :half] ** 2 + g_q[..., half:] ** 2, rtol=1e-12)
    one, zero = np.ones((S, half)), np.zeros((S, half))
    dx0, _, gy0 = orc.qkv_rope_bwd(g_q, g_k, g_v, x, w, one, zero)
    cat = np.concatenate([t.transpose(0, 2, 1, 3).reshape(B, S, -1) for t in (g_q, g_k, g_v)], axis=-1)
    np.testing.assert_allclose(gy0, cat, rtol=0, atol=0)
    np.testing.assert_allclose(dx0, cat @ w, rtol=1e-12, atol=1e-12)

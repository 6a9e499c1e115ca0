"""ctypes front end of the CPU oracle (``attn_ref.c``).

TEST INFRASTRUCTURE ONLY: imported by the test-suite, the smoke check and the
benchmark's cpu-baseline / reference legs.  The CUDA library and its Python
binding never import this module, and this module never imports them.

Every function takes and returns numpy float64 arrays shaped ``[B,H,S,D]``
(``[B,H,S]`` for LSE).  Inputs in f32 or bf16 convert to f64 exactly, so the
caller just passes ``x.double().numpy()``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "attn_ref.c")
_SRC_EXT = os.path.join(_HERE, "attn_ref_ext.c")      # separate query/key lengths, grouped K/V heads
_SRC_PROJ = os.path.join(_HERE, "proj_ref.c")         # output projection of the concatenated heads
_LIB = os.path.join(_HERE, "libmgn_oracle.so")
_lib = None

_dp = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP, no fast-math). Returns the .so path."""
    newest = max(os.path.getmtime(_SRC), os.path.getmtime(_SRC_EXT), os.path.getmtime(_SRC_PROJ))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, _SRC_EXT, _SRC_PROJ, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i, d = ctypes.c_int, ctypes.c_double
        lib.ref_attn_fwd.argtypes = [_dp] * 5 + [i, i, i, i, i, d, i]
        lib.ref_attn_fwd.restype = None
        lib.ref_attn_bwd.argtypes = [_dp] * 9 + [i, i, i, i, i, d, i]
        lib.ref_attn_bwd.restype = None
        lib.ref_attn_head_matrices.argtypes = [_dp] * 7 + [i, i, i, d]
        lib.ref_attn_head_matrices.restype = None
        lib.ref_grads_from_ds.argtypes = [_dp] * 5 + [i, i, d]
        lib.ref_grads_from_ds.restype = None
        lib.ref_attn_fwd_ext.argtypes = [_dp] * 5 + [i] * 7 + [d, i]
        lib.ref_attn_fwd_ext.restype = i
        lib.ref_attn_bwd_ext.argtypes = [_dp] * 9 + [i] * 7 + [d, i]
        lib.ref_attn_bwd_ext.restype = i
        lib.ref_out_proj_fwd.argtypes = [_dp] * 3 + [i] * 5
        lib.ref_out_proj_fwd.restype = None
        lib.ref_out_proj_bwd_data.argtypes = [_dp] * 5 + [i] * 5
        lib.ref_out_proj_bwd_data.restype = None
        lib.ref_out_proj_bwd_weight.argtypes = [_dp] * 3 + [i] * 5
        lib.ref_out_proj_bwd_weight.restype = None
        lib.ref_qkv_rope.argtypes = [_dp] * 7 + [i] * 6
        lib.ref_qkv_rope.restype = None
        lib.ref_qkv_rope_bwd.argtypes = [_dp] * 10 + [i] * 6
        lib.ref_qkv_rope_bwd.restype = None
        lib.ref_max_threads.argtypes = []
        lib.ref_max_threads.restype = i
        _lib = lib
    return _lib


def _c(a: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a: np.ndarray):
    return a.ctypes.data_as(_dp)


def max_threads() -> int:
    return int(_load().ref_max_threads())


def attn_fwd(q, k, v, causal: bool, scale: float, nthreads: int = 0):
    """Returns (O, LSE) in float64."""
    q, k, v = _c(q), _c(k), _c(v)
    B, H, S, D = q.shape
    assert k.shape == q.shape and v.shape == q.shape
    o = np.empty_like(q)
    lse = np.empty((B, H, S), dtype=np.float64)
    _load().ref_attn_fwd(_p(q), _p(k), _p(v), _p(o), _p(lse), B, H, S, D,
                         int(bool(causal)), float(scale), int(nthreads))
    return o, lse


def attn_bwd(q, k, v, d_o, causal: bool, scale: float, nthreads: int = 0):
    """Returns (O, LSE, dQ, dK, dV) in float64; O and LSE are recomputed here."""
    q, k, v, d_o = _c(q), _c(k), _c(v), _c(d_o)
    B, H, S, D = q.shape
    assert k.shape == q.shape and v.shape == q.shape and d_o.shape == q.shape
    o = np.empty_like(q)
    lse = np.empty((B, H, S), dtype=np.float64)
    dq, dk, dv = np.empty_like(q), np.empty_like(q), np.empty_like(q)
    _load().ref_attn_bwd(_p(q), _p(k), _p(v), _p(d_o), _p(o), _p(lse), _p(dq), _p(dk), _p(dv),
                         B, H, S, D, int(bool(causal)), float(scale), int(nthreads))
    return o, lse, dq, dk, dv


def head_matrices(q, k, v, d_o, causal: bool, scale: float):
    """One head ([S,D] inputs): dense P, dP, dS as [S,S] float64 (masked entries 0)."""
    q, k, v, d_o = _c(q), _c(k), _c(v), _c(d_o)
    S, D = q.shape
    P = np.empty((S, S)); dP = np.empty((S, S)); dS = np.empty((S, S))
    _load().ref_attn_head_matrices(_p(q), _p(k), _p(v), _p(d_o), _p(P), _p(dP), _p(dS),
                                   S, D, int(bool(causal)), float(scale))
    return P, dP, dS


def grads_from_ds(dS, q, k, scale: float):
    """One head: (dQ, dK) = (scale dS K, scale dS^T Q)."""
    dS, q, k = _c(dS), _c(q), _c(k)
    S, D = q.shape
    dq = np.empty_like(q); dk = np.empty_like(q)
    _load().ref_grads_from_ds(_p(dS), _p(q), _p(k), _p(dq), _p(dk), S, D, float(scale))
    return dq, dk


def _ext_dims(q, k):
    B, H, Sq, D = q.shape
    Bk, Hkv, Sk, Dk = k.shape
    assert Bk == B and Dk == D and H % Hkv == 0
    return B, H, Hkv, Sq, Sk, D


def attn_fwd_ext(q, k, v, causal: bool, scale: float, nthreads: int = 0):
    """Separate query/key lengths and grouped key/value heads: q [B,H,Sq,D], k, v [B,Hkv,Sk,D].
    Causal masks are aligned bottom-right (key j visible to query i iff j <= i + Sk - Sq).
    Returns (O [B,H,Sq,D], LSE [B,H,Sq]) in float64."""
    q, k, v = _c(q), _c(k), _c(v)
    B, H, Hkv, Sq, Sk, D = _ext_dims(q, k)
    assert v.shape == k.shape
    o = np.empty_like(q)
    lse = np.empty((B, H, Sq), dtype=np.float64)
    rc = _load().ref_attn_fwd_ext(_p(q), _p(k), _p(v), _p(o), _p(lse), B, H, Hkv, Sq, Sk, D,
                                  int(bool(causal)), float(scale), int(nthreads))
    if rc != 0:
        raise ValueError("shapes outside the definition (H % Hkv != 0, or causal with Sq > Sk)")
    return o, lse


def attn_bwd_ext(q, k, v, d_o, causal: bool, scale: float, nthreads: int = 0):
    """Returns (O, LSE, dQ [B,H,Sq,D], dK, dV [B,Hkv,Sk,D]) in float64; O and LSE are recomputed here."""
    q, k, v, d_o = _c(q), _c(k), _c(v), _c(d_o)
    B, H, Hkv, Sq, Sk, D = _ext_dims(q, k)
    assert v.shape == k.shape and d_o.shape == q.shape
    o = np.empty_like(q)
    lse = np.empty((B, H, Sq), dtype=np.float64)
    dq, dk, dv = np.empty_like(q), np.empty_like(k), np.empty_like(k)
    rc = _load().ref_attn_bwd_ext(_p(q), _p(k), _p(v), _p(d_o), _p(o), _p(lse), _p(dq), _p(dk), _p(dv),
                                  B, H, Hkv, Sq, Sk, D, int(bool(causal)), float(scale), int(nthreads))
    if rc != 0:
        raise ValueError("shapes outside the definition (H % Hkv != 0, or causal with Sq > Sk)")
    return o, lse, dq, dk, dv


def out_proj_fwd(o, w):
    """Output projection of the concatenated heads: o [B,H,S,D], w [H*D,E] -> Y [B,S,E], float64."""
    o, w = _c(o), _c(w)
    B, H, S, D = o.shape
    assert w.shape[0] == H * D
    E = w.shape[1]
    y = np.empty((B, S, E), dtype=np.float64)
    _load().ref_out_proj_fwd(_p(o), _p(w), _p(y), B, H, S, D, E)
    return y


def out_proj_bwd(d_y, w, o):
    """Backward of out_proj_fwd: returns (dO [B,H,S,D], delta [B,H,S] = rowsum(dO o O), dW [H*D,E])."""
    d_y, w, o = _c(d_y), _c(w), _c(o)
    B, H, S, D = o.shape
    E = w.shape[1]
    assert w.shape[0] == H * D and d_y.shape == (B, S, E)
    d_o = np.empty_like(o)
    delta = np.empty((B, H, S), dtype=np.float64)
    d_w = np.empty_like(w)
    _load().ref_out_proj_bwd_data(_p(d_y), _p(w), _p(o), _p(d_o), _p(delta), B, H, S, D, E)
    _load().ref_out_proj_bwd_weight(_p(o), _p(d_y), _p(d_w), B, H, S, D, E)
    return d_o, delta, d_w


def qkv_rope(x, w, cos_t, sin_t, H: int, Hkv: int, D: int):
    """Fused query/key/value projection with rotary embedding (rotate-half pairing, caller's angle table):
    x [B,S,E], w [(H+2Hkv)*D, E], cos_t, sin_t [S, D/2] -> (Q [B,H,S,D], K, V [B,Hkv,S,D]), float64."""
    x, w, cos_t, sin_t = _c(x), _c(w), _c(cos_t), _c(sin_t)
    B, S, E = x.shape
    assert w.shape == ((H + 2 * Hkv) * D, E) and cos_t.shape == (S, D // 2) and sin_t.shape == (S, D // 2) and D <= 1024
    q = np.empty((B, H, S, D)); k = np.empty((B, Hkv, S, D)); v = np.empty((B, Hkv, S, D))
    _load().ref_qkv_rope(_p(x), _p(w), _p(cos_t), _p(sin_t), _p(q), _p(k), _p(v), B, S, E, H, Hkv, D)
    return q, k, v


def qkv_rope_bwd(g_q, g_k, g_v, x, w, cos_t, sin_t):
    """Backward of qkv_rope: gradients with respect to the rotated Q [B,H,S,D], K, V [B,Hkv,S,D] ->
    (dX [B,S,E], dW [(H+2Hkv)*D, E], gY [B,S,(H+2Hkv)*D] = the gradient with respect to the unrotated
    projection, heads concatenated query | key | value), float64."""
    g_q, g_k, g_v, x, w, cos_t, sin_t = _c(g_q), _c(g_k), _c(g_v), _c(x), _c(w), _c(cos_t), _c(sin_t)
    B, H, S, D = g_q.shape
    Hkv = g_k.shape[1]
    E = x.shape[2]
    F = (H + 2 * Hkv) * D
    assert g_k.shape == (B, Hkv, S, D) and g_v.shape == (B, Hkv, S, D) and x.shape == (B, S, E) and w.shape == (F, E)
    assert cos_t.shape == (S, D // 2) and sin_t.shape == (S, D // 2)
    gy = np.empty((B, S, F)); dx = np.empty((B, S, E)); dw = np.empty((F, E))
    _load().ref_qkv_rope_bwd(_p(g_q), _p(g_k), _p(g_v), _p(x), _p(w), _p(cos_t), _p(sin_t), _p(gy), _p(dx), _p(dw),
                             B, S, E, H, Hkv, D)
    return dx, dw, gy

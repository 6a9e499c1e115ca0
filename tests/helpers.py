"""Shared test plumbing: run the CUDA path through the C ABI, run the oracle, compare."""
from __future__ import annotations

import numpy as np
import torch

from oracle import attn_oracle as orc
from paper_2608_01563_b200 import binding as mgn

# Gates (strict: f32 FFMA path; fast: bf16 tensor-core path).
STRICT_REL_L2 = 1e-5
STRICT_MAX_ABS = 5e-5
FAST_REL_L2 = 2e-2

GUARD = 64  # canary elements before and after every output buffer


def rel_l2(x: np.ndarray, ref: np.ndarray) -> float:
    den = float(np.linalg.norm(ref.ravel()))
    return float(np.linalg.norm((x - ref).ravel())) / (den if den > 0 else 1.0)


def max_abs(x: np.ndarray, ref: np.ndarray) -> float:
    return float(np.abs(x - ref).max()) if x.size else 0.0


def norm_max_abs(x: np.ndarray, ref: np.ndarray) -> float:
    """max|err| / max(1, max|ref|): equals the literal max-abs whenever the reference is O(1)."""
    return max_abs(x, ref) / max(1.0, float(np.abs(ref).max()) if ref.size else 1.0)


class Guarded:
    """Output buffer with NaN poison inside and canaries on both sides."""

    def __init__(self, shape, dtype, device="cuda"):
        n = int(np.prod(shape))
        self.shape = shape
        self.n = n
        self.buf = torch.full((n + 2 * GUARD,), 512.0, dtype=dtype, device=device)
        self.view = self.buf[GUARD:GUARD + n].view(shape)
        self.view.fill_(float("nan"))
        assert self.view.data_ptr() % 16 == 0

    def check(self, name):
        b = self.buf.float().cpu()
        assert (b[:GUARD] == 512.0).all() and (b[GUARD + self.n:] == 512.0).all(), f"{name}: wrote outside its buffer"
        out = self.view.detach().cpu()
        assert not torch.isnan(out.float()).any(), f"{name}: unwritten or NaN elements"
        return out


def run_cuda(q, k, v, d_o, causal, scale, mode, run_bwd=True, given_o=None, given_lse=None):
    """q,k,v,d_o: host tensors [B,H,S,D] in the mode's dtype. Returns dict of host tensors."""
    dev = "cuda"
    dt = q.dtype
    B, H, S, D = q.shape
    qd, kd, vd, dod = (t.to(dev) for t in (q, k, v, d_o))
    o = Guarded((B, H, S, D), dt)
    lse = Guarded((B, H, S), torch.float32)
    mgn.mgn_attn_fwd(qd, kd, vd, o.view, lse.view, causal, scale, mode)
    res = {}
    if run_bwd:
        dq, dk, dv = (Guarded((B, H, S, D), dt) for _ in range(3))
        ws = mgn.alloc_workspace(B, H, S, D, mode)
        ws.fill_(0xFF)
        o_in = o.view if given_o is None else given_o.to(dev)
        lse_in = lse.view if given_lse is None else given_lse.to(dev)
        mgn.mgn_attn_bwd(qd, kd, vd, o_in, dod, lse_in, dq.view, dk.view, dv.view, ws, causal, scale, mode)
    mgn.mgn_attn_check()
    res["O"] = o.check("O")
    res["LSE"] = lse.check("LSE")
    if run_bwd:
        res["dQ"] = dq.check("dQ")
        res["dK"] = dk.check("dK")
        res["dV"] = dv.check("dV")
    return res


def run_oracle(q, k, v, d_o, causal, scale, heads=None):
    """Oracle on all heads, or on the listed flat (b*H+h) heads -> arrays [1,n,S,D]."""
    B, H, S, D = q.shape

    def prep(t):
        a = t.double().numpy().reshape(1, B * H, S, D)
        return a if heads is None else np.ascontiguousarray(a[:, heads])

    o, lse, dq, dk, dv = orc.attn_bwd(prep(q), prep(k), prep(v), prep(d_o), causal, scale)
    return {"O": o, "LSE": lse, "dQ": dq, "dK": dk, "dV": dv}


def select(res, B, H, heads=None):
    """CUDA results as float64 numpy [1,n,...] restricted to `heads`."""
    out = {}
    for name, t in res.items():
        a = t.double().numpy()
        a = a.reshape(1, B * H, *a.shape[2:])
        out[name] = a if heads is None else np.ascontiguousarray(a[:, heads])
    return out


def check_strict(got, ref, names=("O", "LSE", "dQ", "dK", "dV"), literal_max_abs=True, label=""):
    report = {}
    for n in names:
        r, a, na = rel_l2(got[n], ref[n]), max_abs(got[n], ref[n]), norm_max_abs(got[n], ref[n])
        report[n] = (r, a, na)
        assert r <= STRICT_REL_L2, f"{label}{n}: rel-L2 {r:.3e} > {STRICT_REL_L2}"
        bound = a if literal_max_abs else na
        assert bound <= STRICT_MAX_ABS, f"{label}{n}: max-abs {a:.3e} (normalised {na:.3e}) > {STRICT_MAX_ABS}"
    return report


def check_fast(got, ref, names=("O", "dQ", "dK", "dV"), label=""):
    report = {}
    for n in names:
        r = rel_l2(got[n], ref[n])
        report[n] = r
        assert r <= FAST_REL_L2, f"{label}{n}: rel-L2 {r:.3e} > {FAST_REL_L2}"
    if "LSE" in got:
        r = rel_l2(got["LSE"], ref["LSE"])
        assert r <= 1e-3, f"{label}LSE: rel-L2 {r:.3e}"
    return report


def check_invariants(q, k, v, d_o, res, rtol, max_heads=None):
    """<dQ,Q> = <dK,K> and <dV,V> = <dO,O> per head, evaluated in f64 from the CUDA outputs.
    `max_heads` limits the check to that many evenly spaced heads (host memory at the largest sizes)."""
    if max_heads is not None:
        B, H = q.shape[:2]
        idx = torch.linspace(0, B * H - 1, max_heads).long()
        pick = lambda t: t.reshape(1, B * H, *t.shape[2:])[:, idx]
        q, k, v, d_o = (pick(t) for t in (q, k, v, d_o))
        res = {n: pick(t) for n, t in res.items()}
    f = lambda t: t.double()
    i1a = (f(res["dQ"]) * f(q)).sum(dim=(2, 3))
    i1b = (f(res["dK"]) * f(k)).sum(dim=(2, 3))
    i2a = (f(res["dV"]) * f(v)).sum(dim=(2, 3))
    i2b = (f(d_o) * f(res["O"])).sum(dim=(2, 3))
    # scale of the terms being summed, for a meaningful relative bound
    n1 = (f(res["dQ"]) * f(q)).abs().sum(dim=(2, 3)) + 1e-30
    n2 = (f(res["dV"]) * f(v)).abs().sum(dim=(2, 3)) + 1e-30
    e1 = ((i1a - i1b).abs() / n1).max().item()
    e2 = ((i2a - i2b).abs() / n2).max().item()
    assert e1 <= rtol, f"<dQ,Q> vs <dK,K>: {e1:.3e}"
    assert e2 <= rtol, f"<dV,V> vs <dO,O>: {e2:.3e}"
    return e1, e2


def run_cuda_ext(q, k, v, d_o, causal, scale, mode, run_bwd=True):
    """Extended shapes: q, d_o [B,H,Sq,D]; k, v [B,Hkv,Sk,D] (host tensors). Returns host tensors."""
    dev = "cuda"
    dt = q.dtype
    B, H, Sq, D = q.shape
    _, Hkv, Sk, _ = k.shape
    qd, kd, vd, dod = (t.to(dev) for t in (q, k, v, d_o))
    o = Guarded((B, H, Sq, D), dt)
    lse = Guarded((B, H, Sq), torch.float32)
    mgn.mgn_attn_fwd_ext(qd, kd, vd, o.view, lse.view, causal, scale, mode)
    res = {}
    if run_bwd:
        dq = Guarded((B, H, Sq, D), dt)
        dk, dv = (Guarded((B, Hkv, Sk, D), dt) for _ in range(2))
        ws = mgn.alloc_workspace(B, H, Sq, D, mode)
        ws.fill_(0xFF)
        mgn.mgn_attn_bwd_ext(qd, kd, vd, o.view, dod, lse.view, dq.view, dk.view, dv.view, ws, causal, scale, mode)
    mgn.mgn_attn_check()
    res["O"] = o.check("O")
    res["LSE"] = lse.check("LSE")
    if run_bwd:
        res["dQ"] = dq.check("dQ")
        res["dK"] = dk.check("dK")
        res["dV"] = dv.check("dV")
    return {n: t.double().numpy() for n, t in res.items()}


def run_oracle_ext(q, k, v, d_o, causal, scale):
    o, lse, dq, dk, dv = orc.attn_bwd_ext(q.double().numpy(), k.double().numpy(), v.double().numpy(),
                                          d_o.double().numpy(), causal, scale)
    return {"O": o, "LSE": lse, "dQ": dq, "dK": dk, "dV": dv}

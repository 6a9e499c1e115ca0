"""mgn_attn_bwd_noalloc: the backward entry point for callers that cannot allocate device memory
(plug-ins that are only handed tensors, serving loops where cudaMalloc would stall the GPU).
It must give what mgn_attn_bwd gives -- and what the f64 oracle gives, within the tolerances of
the other parity tests -- call after call, although every call reuses the same built-in scratch
array and finds the previous call's leftovers in it.

Collected last on purpose (file name), so a run that stops at the first failure has already
run every other test."""
import math

import pytest
import torch

from paper_2608_01563_b200 import binding as mgn
from paper_2608_01563_b200 import inputs as synth

import helpers as hp

pytestmark = pytest.mark.gpu


def _forward(q, k, v, causal, scale, mode):
    B, H, S, D = q.shape
    o = torch.empty_like(q)
    lse = torch.empty(B, H, S, device="cuda", dtype=torch.float32)
    mgn.mgn_attn_fwd(q, k, v, o, lse, causal, scale, mode)
    return o, lse


@pytest.mark.parametrize("mode,dtype,gate", [
    (mgn.MODE_STRICT_F32, torch.float32, hp.STRICT_REL_L2),
    (mgn.MODE_FAST_BF16, torch.bfloat16, hp.FAST_REL_L2),
])
def test_noalloc_backward_matches_workspace_backward_twice_in_a_row(mode, dtype, gate):
    # two different problems back to back: the second call meets the first one's scratch contents
    shapes = [(2, 3, 333, 64, True), (1, 4, 200, 128, False)]
    for call, (B, H, S, D, causal) in enumerate(shapes):
        assert mgn.mgn_attn_bwd_workspace_bytes(B, H, S, D, mode) <= mgn.mgn_attn_bwd_noalloc_max_workspace_bytes()
        scale = 1.0 / math.sqrt(D)
        q, k, v, d_o = (t.cuda() for t in synth.random_inputs(500 + call, B, H, S, D, dtype=dtype))
        o, lse = _forward(q, k, v, causal, scale, mode)

        want = [torch.full_like(q, float("nan")) for _ in range(3)]
        ws = mgn.alloc_workspace(B, H, S, D, mode)
        mgn.mgn_attn_bwd(q, k, v, o, d_o, lse, *want, ws, causal, scale, mode)

        got = [torch.full_like(q, float("nan")) for _ in range(3)]
        mgn.mgn_attn_bwd_noalloc(q, k, v, o, d_o, lse, *got, causal, scale, mode)
        mgn.mgn_attn_check()

        for name, g, w in zip(("dQ", "dK", "dV"), got, want):
            g64, w64 = g.double().cpu().numpy(), w.double().cpu().numpy()
            assert not (g64 != g64).any(), f"call {call} {name}: unwritten or NaN elements"
            err = hp.rel_l2(g64, w64)
            assert err <= gate, f"call {call} {name}: rel-L2 {err:.3e} vs the workspace entry point"
            if mode == mgn.MODE_STRICT_F32:
                assert hp.max_abs(g64, w64) <= hp.STRICT_MAX_ABS
        # dK and dV do not depend on accumulation order: identical bits
        assert torch.equal(got[1], want[1]) and torch.equal(got[2], want[2])

        # and against the f64 oracle directly, at the tolerances of the other parity tests
        host = [t.cpu() for t in (q, k, v, d_o)]
        ref = hp.run_oracle(*host, causal, scale)
        mine = hp.select({"dQ": got[0].cpu(), "dK": got[1].cpu(), "dV": got[2].cpu()}, B, H)
        if mode == mgn.MODE_STRICT_F32:
            hp.check_strict(mine, ref, names=("dQ", "dK", "dV"), label=f"noalloc call {call} ")
        else:
            hp.check_fast(mine, ref, names=("dQ", "dK", "dV"), label=f"noalloc call {call} ")


def test_noalloc_rejects_sizes_beyond_its_scratch():
    B, H, S, D = 2, 16, 4096, 128          # fast mode would need ~64 MiB of scratch
    mode = mgn.MODE_FAST_BF16
    assert mgn.mgn_attn_bwd_workspace_bytes(B, H, S, D, mode) > mgn.mgn_attn_bwd_noalloc_max_workspace_bytes()
    t = torch.zeros(16, device="cuda", dtype=torch.bfloat16)     # never dereferenced: the call must refuse first
    lse = torch.zeros(16, device="cuda")
    st = mgn.lib().mgn_attn_bwd_noalloc(*([t.data_ptr()] * 5), lse.data_ptr(), *([t.data_ptr()] * 3),
                                         B, H, S, D, 1, 0.1, mode, None)
    assert st == 4, mgn.mgn_status_string(st)
    # and bad arguments are still named exactly as by mgn_attn_bwd
    st = mgn.lib().mgn_attn_bwd_noalloc(*([t.data_ptr()] * 5), lse.data_ptr(), *([t.data_ptr()] * 3),
                                         1, 1, 8, 48, 0, 0.1, mgn.MODE_STRICT_F32, None)
    assert st == 2, mgn.mgn_status_string(st)

"""Small GPU checks of the library plumbing that the parity files do not cover."""
import pytest
import torch

from paper_2608_01563_b200 import binding as mgn
from paper_2608_01563_b200 import inputs as synth

import helpers as hp

pytestmark = pytest.mark.gpu


def test_measured_ffma_peak_is_plausible():
    t = mgn.mgn_measure_fp32_ffma_tflops()
    # 148 SMs x 128 lanes x 2 x 1.965 GHz = 74.4 TFLOP/s nominal; anything from a throttled to a
    # boosted part should land in this window
    assert 30.0 < t < 90.0, t


def test_profile_events_bracket_the_main_kernels():
    B, H, S, D = 2, 4, 512, 64
    q, k, v, d_o = (t.cuda() for t in synth.random_inputs(3, B, H, S, D))
    o = torch.empty_like(q)
    lse = torch.empty(B, H, S, device="cuda")
    dq, dk, dv = (torch.empty_like(q) for _ in range(3))
    ws = mgn.alloc_workspace(B, H, S, D, mgn.MODE_STRICT_F32)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    for e in ev:
        e.record()
    torch.cuda.synchronize()
    mgn.mgn_attn_profile_events(ev[0].cuda_event, ev[1].cuda_event)
    mgn.mgn_attn_fwd(q, k, v, o, lse, True, 0.125, mgn.MODE_STRICT_F32)
    mgn.mgn_attn_profile_events(ev[2].cuda_event, ev[3].cuda_event)
    mgn.mgn_attn_bwd(q, k, v, o, d_o, lse, dq, dk, dv, ws, True, 0.125, mgn.MODE_STRICT_F32)
    mgn.mgn_attn_profile_events(None, None)
    torch.cuda.synchronize()
    assert ev[0].elapsed_time(ev[1]) > 0.0 and ev[2].elapsed_time(ev[3]) > 0.0
    assert ev[1].elapsed_time(ev[2]) >= 0.0          # forward ends before backward's main kernel starts
    with pytest.raises(mgn.MgnError):
        mgn.mgn_attn_profile_events(ev[0].cuda_event, None)


def test_fast_and_strict_agree_with_each_other():
    """Two independent kernel families on the same (bf16-representable) inputs."""
    B, H, S, D = 1, 2, 384, 128
    q, k, v, d_o = synth.random_inputs(21, B, H, S, D, dtype=torch.bfloat16)
    fast = hp.run_cuda(q, k, v, d_o, True, D ** -0.5, mgn.MODE_FAST_BF16)
    strict = hp.run_cuda(*(t.float() for t in (q, k, v, d_o)), True, D ** -0.5, mgn.MODE_STRICT_F32)
    for name in ("O", "dQ", "dK", "dV"):
        err = hp.rel_l2(fast[name].double().numpy(), strict[name].double().numpy())
        assert err <= hp.FAST_REL_L2, (name, err)
    assert hp.rel_l2(fast["LSE"].double().numpy(), strict["LSE"].double().numpy()) <= 1e-3


def test_check_reports_ok_after_clean_runs():
    mgn.mgn_attn_check()
    assert mgn.mgn_status_string(0) == "MGN_OK"

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


@pytest.mark.parametrize("mode,dtype", [(mgn.MODE_STRICT_F32, torch.float32), (mgn.MODE_FAST_BF16, torch.bfloat16)])
def test_two_host_threads_on_two_streams(mode, dtype):
    """The header allows distinct host threads on distinct streams (the tensor-map cache and the
    per-device set-up are shared state behind a mutex; every call has its own workspace).  Two threads
    run different problems twenty times each; every result must equal what the same call gives alone."""
    import threading
    shapes = [(2, 4, 300, 64, True), (1, 6, 200, 128, False)]
    work = []
    for n, (B, H, S, D, causal) in enumerate(shapes):
        q, k, v, d_o = (t.cuda() for t in synth.random_inputs(60 + n, B, H, S, D, dtype=dtype))
        work.append(dict(q=q, k=k, v=v, d_o=d_o, causal=causal, scale=D ** -0.5, S=S,
                         ws=mgn.alloc_workspace(B, H, S, D, mode), stream=torch.cuda.Stream()))

    def run(w, outs):
        B, H, S, D = w["q"].shape
        o = torch.empty_like(w["q"]); lse = torch.empty(B, H, S, device="cuda")
        dq, dk, dv = (torch.empty_like(w["q"]) for _ in range(3))
        st = w["stream"].cuda_stream
        mgn.mgn_attn_fwd(w["q"], w["k"], w["v"], o, lse, w["causal"], w["scale"], mode, stream=st)
        mgn.mgn_attn_bwd(w["q"], w["k"], w["v"], o, w["d_o"], lse, dq, dk, dv, w["ws"], w["causal"], w["scale"], mode, stream=st)
        outs.append((o, lse, dq, dk, dv))

    torch.cuda.synchronize()
    alone = []
    for w in work:
        outs = []
        run(w, outs)
        w["stream"].synchronize()
        alone.append(outs[0])

    results = [[], []]
    errors = []

    def loop(idx):
        try:
            for _ in range(20):
                run(work[idx], results[idx])
            work[idx]["stream"].synchronize()
        except Exception as exc:                     # surfaces in the main thread below
            errors.append(exc)

    threads = [threading.Thread(target=loop, args=(idx,)) for idx in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    mgn.mgn_attn_check()
    for idx in range(2):
        ref = alone[idx]
        for got in results[idx]:
            for name, g, r in zip(("O", "LSE", "dQ", "dK", "dV"), got, ref):
                if name == "dQ":                     # accumulated with floating-point reductions: order varies
                    assert hp.rel_l2(g.double().cpu().numpy(), r.double().cpu().numpy()) <= (1e-6 if mode == mgn.MODE_STRICT_F32 else 2e-2)
                else:
                    assert torch.equal(g, r), (name, idx, float((g.float() - r.float()).abs().max()), int((g != r).sum()))

#!/usr/bin/env python
"""Benchmark of the attention forward+backward hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload NAME] [--mode strict|fast]

A step is one forward call plus one backward call (preprocess, dQ clear, fused
dK/dV/dQ kernel) over one batch of seeded synthetic input.  Prints ONE JSON line.
The metric is counted GEMM TFLOP/s: forward 4*BH*Np*D, backward 10*BH*Np*D with
Np = S^2 (full) or S^2/2 (causal).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2608_01563_b200 import inputs as synth  # noqa: E402

METRIC = "attention fwd+bwd TFLOP/s per B200 (strict f32, bf16) and % of matching peak"
# dram__bytes_read.sum + dram__bytes_write.sum of the backward main kernel, one launch, as recorded in the
# ncu summary named beside it (same workload and launch configuration as the bench; re-taken when that
# kernel changes -- the record carries the file so that a stale figure can be told)
NCU_TRAFFIC = {
    ("strict", "gpt2_small"): (140.9e6 + 41.3e6, "profiles/strict_fwd_bwd_gpt2_small.md",
                               "strict_bwd_kernel<64,64,64,128,false,true>"),
    ("fast", "long_context"): (203.3e6 + 88.7e6, "profiles/fast_fwd_bwd_long_context.md",
                               "fast_bwd_kernel<128,false,true>"),
}
SM_COUNT = 148
FP32_LANES_PER_SM = 128


def flops(w, which):
    npairs = w.S * w.S / (2.0 if w.causal else 1.0)
    unit = w.BH * npairs * w.D
    return {"fwd": 4.0 * unit, "bwd": 10.0 * unit, "sum": 14.0 * unit}[which]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return json.load(fh), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 1965.0}, "fallback"


def fp32_peak_tflops(peaks):
    """FFMA peak: SMs x 128 lanes x 2 flop x max SM clock."""
    return SM_COUNT * FP32_LANES_PER_SM * 2 * peaks.get("sm_max_mhz", 1965.0) * 1e6 / 1e12


def rank_workload(w, rank):
    """Rank r works on its own batch of the same shape (heads are independent units, so there is
    no data-path collective): same workload, sweep index offset by 1000*r in the seed."""
    import dataclasses
    return dataclasses.replace(w, sweep=w.sweep + 1000 * rank)


def max_over_ranks(values, dist, device):
    """Element-wise MAX over ranks of a list of floats (identity without a process group)."""
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_tflops(w, world, steps, total_ms):
    """Weak scaling: every rank runs the full workload; value = all ranks' counted FLOPs / max time."""
    return world * flops(w, "sum") * steps / (total_ms * 1e-3) / 1e12


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap,timestamp")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.fh = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.fh, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    @staticmethod
    def _epoch(stamp):
        """nvidia-smi's 'YYYY/MM/DD HH:MM:SS.mmm' (local time) as seconds since the epoch."""
        try:
            head, _, ms = stamp.partition(".")
            return time.mktime(time.strptime(head, "%Y/%m/%d %H:%M:%S")) + float("0." + (ms or "0"))
        except ValueError:
            return None

    def stop(self, t_begin=None, t_end=None):
        """Statistics over the samples taken between the two wall-clock times (all samples if none given)."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.fh.close()
        sm, mx, reasons, power = [], [], set(), []
        for line in open(self.path):
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            if t_begin is not None and len(parts) >= 10:
                t = self._epoch(parts[9])
                if t is not None and not (t_begin <= t <= t_end):
                    continue
            try:
                sm.append(float(parts[1])); mx.append(float(parts[2])); power.append(float(parts[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons),
                       samples=len(sm), power_w_max=max(power))
        return out


def quick_measure(mgn, w, mode, dtype, steps, warmup):
    """Device-resident timing of forward and backward calls of one more workload (CUDA events)."""
    q, k, v, d_o = (t.cuda() for t in synth.make_inputs(w, dtype=dtype))
    B, H, S, D = q.shape
    o = torch.empty_like(q)
    lse = torch.empty(B, H, S, device="cuda", dtype=torch.float32)
    dq, dk, dv = (torch.empty_like(q) for _ in range(3))
    ws = mgn.alloc_workspace(B, H, S, D, mode)
    for _ in range(warmup):
        mgn.mgn_attn_fwd(q, k, v, o, lse, w.causal, w.scale, mode)
        mgn.mgn_attn_bwd(q, k, v, o, d_o, lse, dq, dk, dv, ws, w.causal, w.scale, mode)
    torch.cuda.synchronize()
    e = [torch.cuda.Event(enable_timing=True) for _ in range(2 * steps + 1)]
    e[0].record()
    for i in range(steps):
        mgn.mgn_attn_fwd(q, k, v, o, lse, w.causal, w.scale, mode)
        e[2 * i + 1].record()
        mgn.mgn_attn_bwd(q, k, v, o, d_o, lse, dq, dk, dv, ws, w.causal, w.scale, mode)
        e[2 * i + 2].record()
    torch.cuda.synchronize()
    mgn.mgn_attn_check()
    fwd_ms = statistics.mean(e[2 * i].elapsed_time(e[2 * i + 1]) for i in range(steps))
    bwd_ms = statistics.mean(e[2 * i + 1].elapsed_time(e[2 * i + 2]) for i in range(steps))
    return fwd_ms, bwd_ms


def fast_mode_summary(mgn, peaks, gpu_index, steps, warmup):
    """The fast (bf16 tensor-core) mode on its own target workloads, with a clock record of its own:
    long_context timed like the headline (whole calls and the backward main kernel through the
    profile-event hook), then the decoder sweep on its own heavy-tailed inputs.  Compact on purpose:
    it is the last key of the JSON line."""
    wf = synth.WORKLOADS["long_context"]
    mode, dt = mgn.MODE_FAST_BF16, torch.bfloat16
    q, k, v, d_o = (t.cuda() for t in synth.make_inputs(wf, dtype=dt))
    o = torch.empty_like(q)
    lse = torch.empty(wf.B, wf.H, wf.S, device="cuda", dtype=torch.float32)
    dq, dk, dv = (torch.empty_like(q) for _ in range(3))
    ws = mgn.alloc_workspace(wf.B, wf.H, wf.S, wf.D, mode)
    fwd = lambda: mgn.mgn_attn_fwd(q, k, v, o, lse, wf.causal, wf.scale, mode)
    bwd = lambda: mgn.mgn_attn_bwd(q, k, v, o, d_o, lse, dq, dk, dv, ws, wf.causal, wf.scale, mode)
    for _ in range(warmup):
        fwd(); bwd()
    ev = lambda: torch.cuda.Event(enable_timing=True)
    e = [ev() for _ in range(2 * steps + 1)]
    main = [(ev(), ev()) for _ in range(steps)]
    for a, b in main:
        a.record(); b.record()
    torch.cuda.synchronize()
    sampler = ClockSampler(gpu_index)
    sampler.start()
    time.sleep(0.2)
    t0 = time.time()
    e[0].record()
    for i in range(steps):
        fwd()
        e[2 * i + 1].record()
        mgn.mgn_attn_profile_events(main[i][0].cuda_event, main[i][1].cuda_event)
        bwd()
        mgn.mgn_attn_profile_events(None, None)
        e[2 * i + 2].record()
    torch.cuda.synchronize()
    t_cont = time.time()
    while time.time() - t_cont < 0.4:       # keep the same load up until the sampler has seen it
        for _ in range(10):
            fwd(); bwd()
        torch.cuda.synchronize()
    clocks = sampler.stop(t0, time.time())
    mgn.mgn_attn_check()
    f_ms = statistics.median(e[2 * i].elapsed_time(e[2 * i + 1]) for i in range(steps))
    b_ms = statistics.median(e[2 * i + 1].elapsed_time(e[2 * i + 2]) for i in range(steps))
    bm_ms = statistics.median(a.elapsed_time(b) for a, b in main)
    tfl = flops(wf, "sum") / ((f_ms + b_ms) * 1e-3) / 1e12
    out = {"workload": wf.name, "fwd_ms": round(f_ms, 4), "bwd_ms": round(b_ms, 4), "bwd_main_ms": round(bm_ms, 4),
           "sum_tflops": round(tfl, 1), "frac_burst": round(tfl / peaks["bf16_tflops"], 3),
           "frac_sustained": round(tfl / peaks["bf16_tflops_sustained"], 3),
           "clocks": {"sm_mhz": clocks.get("sm_mhz"), "reasons": clocks.get("reasons")}}
    del q, k, v, d_o, o, lse, dq, dk, dv, ws
    sweep = {}
    for name in [n for n in synth.WORKLOADS if n.startswith("decoder_sweep_S")]:
        wt = synth.WORKLOADS[name]
        steps_t = max(2, min(steps, 5 if wt.S <= 2048 else 2))
        fm, bm = quick_measure(mgn, wt, mode, dt, steps_t, 3)
        t = flops(wt, "sum") / ((fm + bm) * 1e-3) / 1e12
        sweep[f"S{wt.S}"] = {"fwd_ms": round(fm, 4), "bwd_ms": round(bm, 4), "sum_tflops": round(t, 1),
                             "frac_burst": round(t / peaks["bf16_tflops"], 3)}
    out["decoder_sweep"] = sweep
    return out


def measure_proj_fusion(mgn, steps, warmup):
    """The output projection at attention's two seams on the long_context shape (E = H*D): this
    library's fused kernels against the unfused sequence (torch's library GEMM plus the layout copy it
    needs, and the attention backward with its own delta pass).  Device-resident, CUDA events."""
    wl = synth.WORKLOADS["long_context"]
    B, H, S, D = wl.B, wl.H, wl.S, wl.D
    E = H * D
    mode, dt = mgn.MODE_FAST_BF16, torch.bfloat16
    q, k, v, _ = (t.cuda() for t in synth.make_inputs(wl, dtype=dt))
    g = torch.Generator(device="cuda").manual_seed(7)
    w = (torch.randn(H * D, E, device="cuda", generator=g) / (H * D) ** 0.5).to(dt)
    d_y = torch.randn(B, S, E, device="cuda", generator=g).to(dt)
    o = torch.empty_like(q); lse = torch.empty(B, H, S, device="cuda")
    mgn.mgn_attn_fwd(q, k, v, o, lse, wl.causal, wl.scale, mode)
    y = torch.empty(B, S, E, device="cuda", dtype=dt)
    d_o = torch.empty_like(q); delta = torch.empty(B, H, S, device="cuda")
    dq, dk, dv = (torch.empty_like(q) for _ in range(3))
    ws = mgn.alloc_workspace(B, H, S, D, mode)

    def timed(fn):
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        e = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        e[0].record()
        for i in range(steps):
            fn()
            e[i + 1].record()
        torch.cuda.synchronize()
        return statistics.median(e[i].elapsed_time(e[i + 1]) for i in range(steps))

    def unfused_fwd():
        torch.matmul(o.transpose(1, 2).reshape(B, S, H * D), w, out=y)

    def unfused_bwd():
        d_o.copy_(torch.matmul(d_y, w.t()).view(B, S, H, D).transpose(1, 2))
        mgn.mgn_attn_bwd(q, k, v, o, d_o, lse, dq, dk, dv, ws, wl.causal, wl.scale, mode)

    def fused_bwd():
        mgn.mgn_out_proj_bwd_data(d_y, w, o, d_o, delta, mode)
        mgn.mgn_attn_bwd_given_delta(q, k, v, d_o, lse, delta, dq, dk, dv, ws, wl.causal, wl.scale, mode)

    # weight gradient and the fused QKV projection with rotary embedding (query/key/value heads = H each)
    d_w = torch.empty_like(w)
    x = torch.randn(B, S, E, device="cuda", generator=g).to(dt)
    w_qkv = (torch.randn(3 * H * D, E, device="cuda", generator=g) / E ** 0.5).to(dt)
    inv = 10000.0 ** (-torch.arange(D // 2, device="cuda", dtype=torch.float32) * 2.0 / D)
    ang = torch.arange(S, device="cuda", dtype=torch.float32)[:, None] * inv[None, :]
    cos_t, sin_t = torch.cos(ang).contiguous(), torch.sin(ang).contiguous()
    q2, k2, v2 = (torch.empty_like(q) for _ in range(3))

    def unfused_dw():
        torch.matmul(o.transpose(1, 2).reshape(B * S, H * D).t(), d_y.view(B * S, E), out=d_w)

    def unfused_qkv():
        yq = torch.matmul(x, w_qkv.t()).view(B, S, 3 * H, D).transpose(1, 2)          # [B, 3H, S, D] view
        c = torch.cat([cos_t, cos_t], dim=1).to(dt)
        s_ = torch.cat([sin_t, sin_t], dim=1).to(dt)
        qk = yq[:, :2 * H]
        rot = torch.cat([-qk[..., D // 2:], qk[..., :D // 2]], dim=-1)
        qk = qk * c + rot * s_
        q2.copy_(qk[:, :H]); k2.copy_(qk[:, H:]); v2.copy_(yq[:, 2 * H:])

    # backward of the QKV projection: opposite rotation of dq, dk, then the data and weight gradients
    gq, gk, gv = (torch.randn(B, H, S, D, device="cuda", generator=g).to(dt) for _ in range(3))
    d_x = torch.empty(B, S, E, device="cuda", dtype=dt)
    d_wqkv = torch.empty_like(w_qkv)

    def fused_qkv_bwd():
        mgn.mgn_rope_bwd_inplace(gq, gk, cos_t, sin_t, mode)
        mgn.mgn_qkv_bwd_data(gq, gk, gv, w_qkv, d_x, mode)
        mgn.mgn_qkv_bwd_weight(gq, gk, gv, x, d_wqkv, mode)

    def unfused_qkv_bwd():
        c = torch.cat([cos_t, cos_t], dim=1).to(dt)
        s_ = torch.cat([sin_t, sin_t], dim=1).to(dt)
        qk = torch.cat([gq, gk], dim=1)
        rot = torch.cat([qk[..., D // 2:], -qk[..., :D // 2]], dim=-1)
        gy = torch.cat([qk * c + rot * s_, gv], dim=1).transpose(1, 2).reshape(B * S, 3 * H * D)
        torch.matmul(gy, w_qkv, out=d_x.view(B * S, E))
        torch.matmul(gy.t(), x.view(B * S, E), out=d_wqkv)

    # a whole attention layer, forward and backward, through this library's entry points only ...
    y2 = torch.empty(B, S, E, device="cuda", dtype=dt)
    d_wo = torch.empty_like(w)

    def layer_fused():
        mgn.mgn_qkv_rope_fwd(x, w_qkv, cos_t, sin_t, q2, k2, v2, mode)
        mgn.mgn_attn_fwd(q2, k2, v2, o, lse, wl.causal, wl.scale, mode)
        mgn.mgn_out_proj_fwd(o, w, y2, mode)
        mgn.mgn_out_proj_bwd_weight(o, d_y, d_wo, mode)
        mgn.mgn_out_proj_bwd_data(d_y, w, o, d_o, delta, mode)
        mgn.mgn_attn_bwd_given_delta(q2, k2, v2, d_o, lse, delta, dq, dk, dv, ws, wl.causal, wl.scale, mode)
        mgn.mgn_rope_bwd_inplace(dq, dk, cos_t, sin_t, mode)
        mgn.mgn_qkv_bwd_data(dq, dk, dv, w_qkv, d_x, mode)
        mgn.mgn_qkv_bwd_weight(dq, dk, dv, x, d_wqkv, mode)

    # ... and the same layer with library GEMMs, eager rotations and layout copies around this library's
    # attention kernels (what a caller without the fused projections would run)
    def layer_unfused():
        unfused_qkv()
        mgn.mgn_attn_fwd(q2, k2, v2, o, lse, wl.causal, wl.scale, mode)
        unfused_fwd()
        unfused_dw()
        d_o.copy_(torch.matmul(d_y, w.t()).view(B, S, H, D).transpose(1, 2))
        mgn.mgn_attn_bwd(q2, k2, v2, o, d_o, lse, dq, dk, dv, ws, wl.causal, wl.scale, mode)
        c = torch.cat([cos_t, cos_t], dim=1).to(dt)
        s_ = torch.cat([sin_t, sin_t], dim=1).to(dt)
        qk = torch.cat([dq, dk], dim=1)
        rot = torch.cat([qk[..., D // 2:], -qk[..., :D // 2]], dim=-1)
        gy = torch.cat([qk * c + rot * s_, dv], dim=1).transpose(1, 2).reshape(B * S, 3 * H * D)
        torch.matmul(gy, w_qkv, out=d_x.view(B * S, E))
        torch.matmul(gy.t(), x.view(B * S, E), out=d_wqkv)

    layer_f = timed(layer_fused)
    layer_u = timed(layer_unfused)
    attn_flops = 14.0 * B * H * (S * S / 2.0) * D if wl.causal else 14.0 * B * H * S * S * D
    layer_flops = attn_flops + 2.0 * B * S * E * (3 * H * D) * 3 + 2.0 * B * S * (H * D) * E * 3

    gemm_flops = 2.0 * B * S * H * D * E
    qb_fused = timed(fused_qkv_bwd)
    qb_unf = timed(unfused_qkv_bwd)
    w_fused = timed(lambda: mgn.mgn_out_proj_bwd_weight(o, d_y, d_w, mode))
    w_unf = timed(unfused_dw)
    qkv_fused = timed(lambda: mgn.mgn_qkv_rope_fwd(x, w_qkv, cos_t, sin_t, q2, k2, v2, mode))
    qkv_unf = timed(unfused_qkv)
    f_fused = timed(lambda: mgn.mgn_out_proj_fwd(o, w, y, mode))
    f_unf = timed(unfused_fwd)
    p_fused = timed(lambda: mgn.mgn_out_proj_bwd_data(d_y, w, o, d_o, delta, mode))
    b_fused = timed(fused_bwd)
    b_unf = timed(unfused_bwd)
    mgn.mgn_attn_check()
    return {"shape": {"B": B, "H": H, "S": S, "D": D, "E": E},
            "out_proj_fwd_ms": {"fused": round(f_fused, 4), "library_gemm_plus_layout_copy": round(f_unf, 4)},
            "out_proj_fwd_tflops": round(gemm_flops / (f_fused * 1e-3) / 1e12, 1),
            "weight_grad_ms": {"fused": round(w_fused, 4), "library_gemm_plus_layout_copy": round(w_unf, 4)},
            "qkv_rope_ms": {"fused": round(qkv_fused, 4), "library_gemm_plus_eager_rotation_and_copies": round(qkv_unf, 4)},
            "qkv_rope_tflops": round(3 * gemm_flops / (qkv_fused * 1e-3) / 1e12, 1),
            "qkv_bwd_ms": {"fused": round(qb_fused, 4), "library_gemms_plus_eager_rotation_and_copies": round(qb_unf, 4)},
            "qkv_bwd_tflops": round(6 * gemm_flops / (qb_fused * 1e-3) / 1e12, 1),
            "layer_fwd_bwd_ms": {"fused": round(layer_f, 4), "library_gemms_eager_rotation_copies_plus_attn": round(layer_u, 4)},
            "layer_fwd_bwd_tflops": round(layer_flops / (layer_f * 1e-3) / 1e12, 1),
            "do_producer_ms": round(p_fused, 4), "do_producer_tflops": round(gemm_flops / (p_fused * 1e-3) / 1e12, 1),
            "proj_bwd_plus_attn_bwd_ms": {"fused": round(b_fused, 4), "library_gemm_plus_layout_copy_plus_attn_bwd": round(b_unf, 4)}}


def quick_measure_ext(mgn, w, mode, dtype, steps, warmup):
    """Device-resident timing of one cross-attention / grouped-head workload (CUDA events)."""
    q, k, v, d_o = (t.cuda() for t in synth.make_inputs_ext(w, dtype=dtype))
    o = torch.empty_like(q)
    lse = torch.empty(w.B, w.H, w.Sq, device="cuda", dtype=torch.float32)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    ws = mgn.alloc_workspace(w.B, w.H, w.Sq, w.D, mode)
    for _ in range(warmup):
        mgn.mgn_attn_fwd_ext(q, k, v, o, lse, w.causal, w.scale, mode)
        mgn.mgn_attn_bwd_ext(q, k, v, o, d_o, lse, dq, dk, dv, ws, w.causal, w.scale, mode)
    torch.cuda.synchronize()
    e = [torch.cuda.Event(enable_timing=True) for _ in range(2 * steps + 1)]
    e[0].record()
    for i in range(steps):
        mgn.mgn_attn_fwd_ext(q, k, v, o, lse, w.causal, w.scale, mode)
        e[2 * i + 1].record()
        mgn.mgn_attn_bwd_ext(q, k, v, o, d_o, lse, dq, dk, dv, ws, w.causal, w.scale, mode)
        e[2 * i + 2].record()
    torch.cuda.synchronize()
    mgn.mgn_attn_check()
    fwd_ms = statistics.mean(e[2 * i].elapsed_time(e[2 * i + 1]) for i in range(steps))
    bwd_ms = statistics.mean(e[2 * i + 1].elapsed_time(e[2 * i + 2]) for i in range(steps))
    unit = w.B * w.H * w.pairs * w.D
    return {"B": w.B, "H": w.H, "H_kv": w.Hkv, "S_q": w.Sq, "S_k": w.Sk, "D": w.D, "causal": w.causal,
            "fwd_ms": fwd_ms, "bwd_ms": bwd_ms, "fwd_tflops": 4.0 * unit / (fwd_ms * 1e-3) / 1e12,
            "bwd_tflops": 10.0 * unit / (bwd_ms * 1e-3) / 1e12,
            "sum_tflops": 14.0 * unit / ((fwd_ms + bwd_ms) * 1e-3) / 1e12}


def measure_deterministic_bwd(mgn, w, mode, dtype, steps, warmup):
    """The backward without floating-point atomics (fused dK+dV kernel + separate dQ pass)."""
    q, k, v, d_o = (t.cuda() for t in synth.make_inputs(w, dtype=dtype))
    o = torch.empty_like(q)
    lse = torch.empty(w.B, w.H, w.S, device="cuda", dtype=torch.float32)
    dq, dk, dv = (torch.empty_like(q) for _ in range(3))
    ws = mgn.alloc_workspace(w.B, w.H, w.S, w.D, mode)
    mgn.mgn_attn_fwd(q, k, v, o, lse, w.causal, w.scale, mode)
    run = lambda: mgn.mgn_attn_bwd_deterministic(q, k, v, o, d_o, lse, dq, dk, dv, ws, w.causal, w.scale, mode)
    for _ in range(warmup):
        run()
    torch.cuda.synchronize()
    e = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    e[0].record()
    for i in range(steps):
        run()
        e[i + 1].record()
    torch.cuda.synchronize()
    mgn.mgn_attn_check()
    ms = statistics.mean(e[i].elapsed_time(e[i + 1]) for i in range(steps))
    return {"workload": w.name, "bwd_ms": ms, "counted_tflops": flops(w, "bwd") / (ms * 1e-3) / 1e12,
            "executed_tflops": 1.4 * flops(w, "bwd") / (ms * 1e-3) / 1e12,
            "note": "no floating-point atomics; 7 matrix products per tile pair instead of 5"}


def measure_accel_policy(mgn, w, steps, warmup):
    """The paper's accelerated policy on f32 tensors: f16 tensor-core forward (mgn_attn_fwd_accel, its
    f32->f16 conversion included) followed by the strict f32 backward."""
    S32 = mgn.MODE_STRICT_F32
    q, k, v, d_o = (t.cuda() for t in synth.make_inputs(w, dtype=torch.float32))
    o = torch.empty_like(q)
    lse = torch.empty(w.B, w.H, w.S, device="cuda", dtype=torch.float32)
    dq, dk, dv = (torch.empty_like(q) for _ in range(3))
    ws = mgn.alloc_workspace(w.B, w.H, w.S, w.D, S32)
    wsf = torch.empty(mgn.mgn_attn_fwd_accel_workspace_bytes(w.B, w.H, w.H, w.S, w.S, w.D), dtype=torch.uint8,
                      device="cuda")
    fwd = lambda: mgn.mgn_attn_fwd_accel(q, k, v, o, lse, wsf, w.causal, w.scale)
    bwd = lambda: mgn.mgn_attn_bwd(q, k, v, o, d_o, lse, dq, dk, dv, ws, w.causal, w.scale, S32)
    for _ in range(warmup):
        fwd()
        bwd()
    torch.cuda.synchronize()
    e = [torch.cuda.Event(enable_timing=True) for _ in range(2 * steps + 1)]
    e[0].record()
    for i in range(steps):
        fwd()
        e[2 * i + 1].record()
        bwd()
        e[2 * i + 2].record()
    torch.cuda.synchronize()
    mgn.mgn_attn_check()
    f_ms = statistics.mean(e[2 * i].elapsed_time(e[2 * i + 1]) for i in range(steps))
    b_ms = statistics.mean(e[2 * i + 1].elapsed_time(e[2 * i + 2]) for i in range(steps))
    return {"workload": w.name, "fwd_ms": f_ms, "bwd_ms": b_ms,
            "fwd_tflops": flops(w, "fwd") / (f_ms * 1e-3) / 1e12,
            "sum_tflops": flops(w, "sum") / ((f_ms + b_ms) * 1e-3) / 1e12,
            "note": "f32 tensors; forward: f32->f16 conversion + f16 tensor-core kernel, f32 O; backward: strict f32"}


def cpu_info():
    model = "unknown"
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                model = line.split(":", 1)[1].strip()
                break
    except OSError:
        pass
    return model


_oracle_inputs = {}
_oracle_outputs = {}


def time_oracle(w, dtype, heads, repeats=1):
    """Oracle forward+backward on the first `heads` heads. Returns (seconds fwd, seconds bwd, threads)."""
    from oracle import attn_oracle as orc
    key = (w.name, w.sweep, dtype, heads)
    if key not in _oracle_inputs:
        _oracle_inputs.clear()
        _oracle_outputs.clear()
        _oracle_inputs[key] = [t.double().numpy() for t in synth.make_inputs(w, dtype=dtype, heads=heads)]
    a = _oracle_inputs[key]
    best_f = best_b = float("inf")
    for _ in range(repeats):
        t0 = time.perf_counter()
        orc.attn_fwd(a[0], a[1], a[2], w.causal, w.scale)
        t1 = time.perf_counter()
        _oracle_outputs[key] = orc.attn_bwd(a[0], a[1], a[2], a[3], w.causal, w.scale)
        t2 = time.perf_counter()
        best_f, best_b = min(best_f, t1 - t0), min(best_b, t2 - t1)
    return best_f, best_b, orc.max_threads()


def parity_figures(w, dtype, heads, gpu_outputs):
    """Per-tensor error of the timed workload's CUDA outputs against the oracle's outputs on the head
    subset the cpu_baseline leg has just computed: rel-L2, the literal max-abs and the max-abs relative to
    max(1, max|ref|) (the strict gate's form on the heavy-tailed decoder sweep)."""
    import numpy as np
    ref = _oracle_outputs.get((w.name, w.sweep, dtype, heads))
    if ref is None:
        return None
    out = {"heads": f"first {heads} of {w.BH}"}
    for name, got, want in zip(("O", "LSE", "dQ", "dK", "dV"), gpu_outputs, ref):
        g = got.reshape(1, w.BH, *got.shape[2:])[:, :heads].double().cpu().numpy()
        err = np.abs(g - want)
        den = float(np.linalg.norm(want.ravel()))
        out[name] = {"rel_l2": float(np.linalg.norm((g - want).ravel())) / (den if den > 0 else 1.0),
                     "max_abs": float(err.max()),
                     "max_abs_normalised": float(err.max()) / max(1.0, float(np.abs(want).max()))}
    return out


def cpu_baseline(w, dtype, budget_s=15.0):
    """The oracle, as it stands, on a bounded head subset sized for ~budget_s of CPU work."""
    from oracle import attn_oracle as orc
    threads = orc.max_threads()
    probe_heads = min(w.BH, threads)
    tf, tb, _ = time_oracle(w, dtype, probe_heads)
    per_round = tf + tb
    rounds = max(1, int(budget_s / max(per_round, 1e-3)))
    heads = min(w.BH, probe_heads * rounds)
    if heads > probe_heads:
        tf, tb, _ = time_oracle(w, dtype, heads)
    # if even all heads take well under the budget, repeat the pass so that about 10 s of CPU work is timed
    passes = max(1, min(50, int(10.0 / max(tf + tb, 1e-3))))
    if passes > 1:
        acc_f = acc_b = 0.0
        for _ in range(passes):
            f1, b1, _ = time_oracle(w, dtype, heads)
            acc_f += f1
            acc_b += b1
        tf, tb = acc_f / passes, acc_b / passes
    fl = flops(w, "sum") * heads / w.BH
    return {"value": fl / (tf + tb) / 1e12, "unit": "TFLOP/s", "cores": threads, "kind": "oracle",
            "sample": (f"first {heads} of {w.BH} heads of {w.name}, mean of {passes} passes "
                       f"(f64, fwd {tf:.2f} s + bwd {tb:.2f} s per pass)"),
            "cpu_model": cpu_info(), "heads": heads}


def run_reference(args, w, dtype):
    """--impl reference: the CPU oracle timed on a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import attn_oracle as orc
    threads = orc.max_threads()
    heads = min(w.BH, threads)
    for _ in range(args.warmup):
        time_oracle(w, dtype, heads)
    times = []
    for _ in range(args.steps):
        tf, tb, _ = time_oracle(w, dtype, heads)
        times.append(tf + tb)
    total = sum(times)
    fl = flops(w, "sum") * heads / w.BH
    value = fl * args.steps / total / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "S": w.S, "D": w.D, "causal": w.causal,
                   "mode": args.mode, "sample_heads": heads},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": threads, "kind": "oracle",
                         "sample": f"first {heads} of {w.BH} heads of {w.name} per step", "cpu_model": cpu_info()},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None)
    ap.add_argument("--mode", default="strict", choices=["strict", "fast"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-fast", action="store_true", help="skip the extra measurements (other mode, other shapes, other workloads)")
    ap.add_argument("--only-proj", action="store_true",
                    help="time only the projections either side of attention (the proj_fusion object of the line) and print "
                         "that object; a small command to capture their kernels under a profiler")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    default_wl = "gpt2_small" if args.mode == "strict" else "long_context"
    w = synth.WORKLOADS[args.workload or default_wl]
    dtype = torch.float32 if args.mode == "strict" else torch.bfloat16

    if args.impl == "reference":
        run_reference(args, w, dtype)
        return

    from paper_2608_01563_b200 import binding as mgn

    if args.only_proj:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the projections have no CPU fallback")
        if int(os.environ.get("RANK", "0")) == 0:
            print(json.dumps({"proj_fusion": measure_proj_fusion(mgn, args.steps, args.warmup)}))
        return

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    mode = mgn.MODE_STRICT_F32 if args.mode == "strict" else mgn.MODE_FAST_BF16

    # Each rank works on its own batch of the same shape (heads are independent units:
    # no data-path collective).  Rank r draws sweep index r*1000 more than rank 0.
    w_rank = rank_workload(w, rank)
    host = [t.pin_memory() for t in synth.make_inputs(w_rank, dtype=dtype)]
    dev = [t.cuda(non_blocking=True) for t in host]
    qd, kd, vd, dod = dev
    B, H, S, D = qd.shape
    o = torch.empty_like(qd)
    lse = torch.empty(B, H, S, device="cuda", dtype=torch.float32)
    dq, dk, dv = (torch.empty_like(qd) for _ in range(3))
    ws = mgn.alloc_workspace(B, H, S, D, mode)
    host_out = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in (o, lse, dq, dk, dv)]
    torch.cuda.synchronize()

    def step():
        mgn.mgn_attn_fwd(qd, kd, vd, o, lse, w.causal, w.scale, mode)
        mgn.mgn_attn_bwd(qd, kd, vd, o, dod, lse, dq, dk, dv, ws, w.causal, w.scale, mode)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    mgn.mgn_attn_check()

    K = args.steps
    ev = lambda: torch.cuda.Event(enable_timing=True)
    e_step0, e_step1 = ev(), ev()
    pairs = {name: [(ev(), ev()) for _ in range(K)] for name in ("fwd_main", "bwd_main")}
    e_fwd_end = [ev() for _ in range(K)]
    for lst in pairs.values():          # create the underlying CUDA events
        for a, b in lst:
            a.record(); b.record()
    torch.cuda.synchronize()

    gpu_index = local_rank
    try:
        gpu_index = int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local_rank])
    except (KeyError, ValueError, IndexError):
        pass
    sampler = ClockSampler(gpu_index)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    t_load0 = time.time()
    e_step0.record()
    for i in range(K):
        a, b = pairs["fwd_main"][i]
        mgn.mgn_attn_profile_events(a.cuda_event, b.cuda_event)
        mgn.mgn_attn_fwd(qd, kd, vd, o, lse, w.causal, w.scale, mode)
        e_fwd_end[i].record()
        a, b = pairs["bwd_main"][i]
        mgn.mgn_attn_profile_events(a.cuda_event, b.cuda_event)
        mgn.mgn_attn_bwd(qd, kd, vd, o, dod, lse, dq, dk, dv, ws, w.causal, w.scale, mode)
    e_step1.record()
    mgn.mgn_attn_profile_events(None, None)
    # The timed region lasts tens of milliseconds, about one sampling period: the same step loop keeps
    # running (untimed) for a little longer so that the clock record holds samples taken under this load.
    barrier()
    t_cont = time.time()
    while time.time() - t_cont < 0.4:
        for _ in range(10):
            step()
        torch.cuda.synchronize()
    t_load1 = time.time()
    clocks = sampler.stop(t_load0, t_load1) if rank == 0 else None
    if clocks is not None:
        clocks["window"] = "samples between the start of the timed region and the end of a 0.4 s continuation of the same step loop"
    mgn.mgn_attn_check()

    total_ms = e_step0.elapsed_time(e_step1)
    fwd_main_ms = statistics.mean(a.elapsed_time(b) for a, b in pairs["fwd_main"])
    bwd_main_ms = statistics.mean(a.elapsed_time(b) for a, b in pairs["bwd_main"])
    # forward call = its one kernel; backward call = everything from the end of forward to the end of the step
    fwd_call_ms = fwd_main_ms
    bwd_call_ms = total_ms / K - fwd_call_ms

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region ----------
    e2e = None
    if not args.no_e2e:
        # The step is pipelined over batch chunks on three streams (host->device, compute,
        # device->host), as a caller of a stream-ordered C ABI would do: every byte still crosses
        # PCIe inside the timed region, but copies overlap the kernels of neighbouring chunks.
        n_chunks = 4 if B % 4 == 0 else (2 if B % 2 == 0 else 1)
        bc = B // n_chunks
        s_cmp = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        ws_c = [mgn.alloc_workspace(bc, H, S, D, mode) for _ in range(n_chunks)]
        in_done = [torch.cuda.Event() for _ in range(n_chunks)]
        cmp_done = [torch.cuda.Event() for _ in range(n_chunks)]
        out_done = [torch.cuda.Event() for _ in range(n_chunks)]
        outs_dev = (o, lse, dq, dk, dv)
        for evt in cmp_done + out_done:
            evt.record(s_cmp)

        def e2e_step():
            for c in range(n_chunks):
                sl = slice(c * bc, (c + 1) * bc)
                with torch.cuda.stream(s_in):
                    s_in.wait_event(cmp_done[c])          # previous step's kernels are done with this chunk's inputs
                    for h, d in zip(host, dev):
                        d[sl].copy_(h[sl], non_blocking=True)
                    in_done[c].record(s_in)
                s_cmp.wait_event(in_done[c])
                s_cmp.wait_event(out_done[c])             # previous step's outputs of this chunk have left the device
                mgn.mgn_attn_fwd(qd[sl], kd[sl], vd[sl], o[sl], lse[sl], w.causal, w.scale, mode)
                mgn.mgn_attn_bwd(qd[sl], kd[sl], vd[sl], o[sl], dod[sl], lse[sl], dq[sl], dk[sl], dv[sl], ws_c[c],
                                 w.causal, w.scale, mode)
                cmp_done[c].record(s_cmp)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(cmp_done[c])
                    for h, d in zip(host_out, outs_dev):
                        h[sl].copy_(d[sl], non_blocking=True)
                    out_done[c].record(s_out)

        def e2e_drain():
            for c in range(n_chunks):
                s_cmp.wait_event(out_done[c])             # the last bytes of the last step are on the host
        # Steps follow each other like the iterations of a training loop: chunk c of the next step may be
        # copied in and computed while later chunks of this step are still leaving the device (each chunk's
        # buffers are guarded by the events above); the timed region ends when the last step's outputs have landed.
        for _ in range(3):
            e2e_step()
        e2e_drain()
        barrier()
        e0, e1 = ev(), ev()
        e0.record()
        for _ in range(K):
            e2e_step()
        e2e_drain()
        e1.record()
        barrier()
        e2e_ms = e0.elapsed_time(e1)
    else:
        e2e_ms = None

    total_ms_max, e2e_ms_max = max_over_ranks([total_ms, e2e_ms or 0.0], dist, "cuda")

    if rank == 0:
        peaks, peak_src = measured_peaks()
        fl_sum = flops(w, "sum")
        value = whole_job_tflops(w, world, K, total_ms_max)
        if args.mode == "strict":
            peak = fp32_peak_tflops(peaks)
            bound = "alu"
            peak_note = f"{SM_COUNT} SMs x {FP32_LANES_PER_SM} FP32 lanes x 2 x {peaks.get('sm_max_mhz', 1965.0):.0f} MHz"
        else:
            peak = peaks["bf16_tflops"]
            bound = "tensor"
            peak_note = (f"{peak_src} dense bf16, burst figure (steps are ~1 ms bursts); "
                         f"sustained {peaks['bf16_tflops_sustained']}")
        bwd_main_tflops = flops(w, "bwd") / (bwd_main_ms * 1e-3) / 1e12
        fwd_main_tflops = flops(w, "fwd") / (fwd_main_ms * 1e-3) / 1e12
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": K,
            "warmup": args.warmup, "ms_per_step": total_ms_max / K, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if args.mode == "strict" else "bf16", "data": "synthetic",
            "config": {"workload": w.name, "B": w.B, "H": w.H, "S": w.S, "D": w.D, "causal": w.causal,
                       "mode": args.mode, "per_rank_batch": "full workload on every rank",
                       "e2e": "pinned host buffers; batch split in chunks pipelined over H2D / compute / D2H streams",
                       "l2": "no flush: Q,K,V,dO,O,dQ,dK,dV of one step exceed the 126 MB L2"
                       if 8 * qd.numel() * qd.element_size() > 126e6 else "working set fits L2 (compute-bound path)"},
            "frac_of_peak": value / world / peak, "peak_tflops": peak, "peak_note": peak_note,
            "fwd_tflops": flops(w, "fwd") / (fwd_call_ms * 1e-3) / 1e12,
            "bwd_tflops": flops(w, "bwd") / (bwd_call_ms * 1e-3) / 1e12,
            "fwd_ms": fwd_call_ms, "bwd_ms": bwd_call_ms,
            "roofline": {"kernel": "bwd_main (fused dK/dV/dQ)", "bound": bound, "achieved": bwd_main_tflops,
                         "peak": peak, "unit": "TFLOP/s", "frac": bwd_main_tflops / peak,
                         "traffic": NCU_TRAFFIC.get((args.mode, w.name), (None,))[0],
                         "traffic_unit": "bytes per launch (ncu dram read+write)",
                         "traffic_source": list(NCU_TRAFFIC.get((args.mode, w.name), (None, None, None))[1:]),
                         "algorithmic_bytes": w.BH * w.S * (8 * w.D * qd.element_size() + 8),
                         "ms_per_launch": bwd_main_ms, "peak_source": peak_note,
                         "fwd_kernel": {"achieved": fwd_main_tflops, "frac": fwd_main_tflops / peak,
                                        "ms_per_launch": fwd_main_ms}},
            "gpu_launches": (3 if args.mode == "strict" else 4) * K,
            "clocks": clocks,
        }
        if e2e_ms is not None:
            h2d = sum(t_.numel() * t_.element_size() for t_ in host)
            d2h = sum(t_.numel() * t_.element_size() for t_ in host_out)
            line["e2e"] = {"value": whole_job_tflops(w, world, K, e2e_ms_max), "unit": "TFLOP/s",
                           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
        if args.mode == "strict":
            measured = mgn.mgn_measure_fp32_ffma_tflops()
            line["fp32_ffma_measured_tflops"] = measured
            line["frac_of_measured_ffma_peak"] = value / world / measured if measured > 0 else None
        if world == 1 and args.workload is None and not args.no_fast:
            # cross-attention and grouped key/value heads (mgn_attn_*_ext), in this run's arithmetic mode
            mode_peak = peak if args.mode == "strict" else peaks["bf16_tflops"]
            ext = {}
            for name in ("gqa_decoder", "gqa_suffix", "cross_attn_text", "cross_attn_action"):
                r = quick_measure_ext(mgn, synth.EXT_WORKLOADS[name], mode, dtype, K, args.warmup)
                r["frac_of_peak"] = r["sum_tflops"] / mode_peak
                ext[name] = r
            line["ext_shapes"] = ext
            # the other configured workloads in this run's arithmetic mode (few steps each): the ragged
            # vision-transformer shape (strict) and the decoder sweep, device-resident like `value`
            names = (["vit_b_ragged"] if args.mode == "strict" else []) + \
                    [n for n in synth.WORKLOADS if n.startswith("decoder_sweep_S")]
            table = {}
            for name in names:
                wt = synth.WORKLOADS[name]
                steps_t = max(2, min(K, 5 if wt.S <= 2048 else 2))
                f_ms, b_ms = quick_measure(mgn, wt, mode, dtype, steps_t, 2)
                tfl = flops(wt, "sum") / ((f_ms + b_ms) * 1e-3) / 1e12
                table[name] = {"B": wt.B, "H": wt.H, "S": wt.S, "D": wt.D, "causal": bool(wt.causal), "steps": steps_t,
                               "fwd_ms": f_ms, "bwd_ms": b_ms,
                               "fwd_tflops": flops(wt, "fwd") / (f_ms * 1e-3) / 1e12,
                               "bwd_tflops": flops(wt, "bwd") / (b_ms * 1e-3) / 1e12,
                               "sum_tflops": tfl, "frac_of_peak": tfl / mode_peak}
            line["other_workloads"] = table
            line["deterministic_bwd"] = measure_deterministic_bwd(mgn, w, mode, dtype, K, args.warmup)
            line["proj_fusion"] = measure_proj_fusion(mgn, K, args.warmup)
            if args.mode == "strict":
                if w.D in (64, 128):
                    line["accel_policy"] = measure_accel_policy(mgn, w, K, args.warmup)
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(w, dtype)
            # error of the timed workload's outputs against the oracle outputs that leg has just produced
            line["parity"] = parity_figures(w, dtype, line["cpu_baseline"].pop("heads"), (o, lse, dq, dk, dv))
        if world == 1 and args.mode == "strict" and args.workload is None and not args.no_fast:
            # The other arithmetic mode of the same library on its own target workloads.  Last key of
            # the line, and compact, so that a reader who keeps only the end of the line still has it.
            line["fast_mode"] = fast_mode_summary(mgn, peaks, gpu_index, K, args.warmup)
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

"""Thin ctypes binding of ``libmgn_attn.so``: argument marshalling only.

Every function mirrors the C entry point of the same name (``include/mgn_attn.h``),
takes torch CUDA tensors for the device buffers and enqueues on the current torch
stream unless ``stream`` (a raw ``cudaStream_t`` integer) is given.  There is no
fallback: if the library has not been built the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

MODE_STRICT_F32 = 0
MODE_FAST_BF16 = 1

MGN_OK = 0
STATUS_NAMES = {
    0: "MGN_OK", 1: "MGN_ERR_INVALID_ARG", 2: "MGN_ERR_UNSUPPORTED", 3: "MGN_ERR_MISALIGNED",
    4: "MGN_ERR_WORKSPACE", 5: "MGN_ERR_CUDA", 6: "MGN_ERR_ARCH", 7: "MGN_ERR_DEVICE_TIMEOUT",
}

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libmgn_attn.so")
_lib = None


class MgnError(RuntimeError):
    def __init__(self, status: int, where: str):
        super().__init__(f"{where} failed: {STATUS_NAMES.get(status, status)}")
        self.status = status


def lib() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it is missing (no CPU or eager fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2608_01563_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
        L.mgn_attn_fwd.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, f, i, vp]
        L.mgn_attn_fwd.restype = i
        L.mgn_attn_bwd.argtypes = [vp] * 9 + [vp, sz, i, i, i, i, i, f, i, vp]
        L.mgn_attn_bwd.restype = i
        L.mgn_attn_fwd_ext.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, i, f, i, vp]
        L.mgn_attn_fwd_ext.restype = i
        L.mgn_attn_bwd_ext.argtypes = [vp] * 9 + [vp, sz, i, i, i, i, i, i, i, f, i, vp]
        L.mgn_attn_bwd_ext.restype = i
        L.mgn_attn_fwd_accel.argtypes = [vp] * 5 + [vp, sz, i, i, i, i, i, i, i, f, vp]
        L.mgn_attn_fwd_accel.restype = i
        L.mgn_attn_fwd_accel_workspace_bytes.argtypes = [i] * 6
        L.mgn_attn_fwd_accel_workspace_bytes.restype = sz
        L.mgn_attn_bwd_deterministic.argtypes = [vp] * 9 + [vp, sz, i, i, i, i, i, i, i, f, i, vp]
        L.mgn_attn_bwd_deterministic.restype = i
        L.mgn_attn_bwd_workspace_bytes.argtypes = [i, i, i, i, i]
        L.mgn_attn_bwd_workspace_bytes.restype = sz
        L.mgn_attn_check.argtypes = [vp]
        L.mgn_attn_check.restype = i
        L.mgn_attn_bwd_noalloc.argtypes = [vp] * 9 + [i, i, i, i, i, f, i, vp]
        L.mgn_attn_bwd_noalloc.restype = i
        L.mgn_attn_bwd_noalloc_max_workspace_bytes.argtypes = []
        L.mgn_attn_bwd_noalloc_max_workspace_bytes.restype = sz
        L.mgn_measure_fp32_ffma_tflops.argtypes = [vp, ctypes.POINTER(ctypes.c_double), vp]
        L.mgn_measure_fp32_ffma_tflops.restype = i
        L.mgn_attn_profile_events.argtypes = [vp, vp]
        L.mgn_attn_profile_events.restype = i
        L.mgn_attn_fast_item_order.argtypes = [i]
        L.mgn_attn_fast_item_order.restype = i
        L.mgn_attn_strict_tiles.argtypes = [i] * 7 + [ctypes.POINTER(ctypes.c_int)]
        L.mgn_attn_strict_tiles.restype = i
        L.mgn_out_proj_fwd.argtypes = [vp, vp, vp, i, i, i, i, i, i, vp]
        L.mgn_out_proj_fwd.restype = i
        L.mgn_out_proj_bwd_data.argtypes = [vp] * 5 + [i, i, i, i, i, i, vp]
        L.mgn_out_proj_bwd_data.restype = i
        L.mgn_out_proj_bwd_weight.argtypes = [vp, vp, vp, i, i, i, i, i, i, vp]
        L.mgn_out_proj_bwd_weight.restype = i
        L.mgn_qkv_rope_fwd.argtypes = [vp] * 7 + [i] * 7 + [vp]
        L.mgn_qkv_rope_fwd.restype = i
        L.mgn_rope_bwd_inplace.argtypes = [vp] * 4 + [i] * 6 + [vp]
        L.mgn_rope_bwd_inplace.restype = i
        L.mgn_qkv_bwd_data.argtypes = [vp] * 5 + [i] * 7 + [vp]
        L.mgn_qkv_bwd_data.restype = i
        L.mgn_qkv_bwd_weight.argtypes = [vp] * 5 + [i] * 7 + [vp]
        L.mgn_qkv_bwd_weight.restype = i
        L.mgn_attn_bwd_given_delta.argtypes = [vp] * 9 + [vp, sz, i, i, i, i, i, i, i, f, i, vp]
        L.mgn_attn_bwd_given_delta.restype = i
        L.mgn_selftest_wait_timeout.argtypes = [vp, vp]
        L.mgn_selftest_wait_timeout.restype = i
        L.mgn_status_string.argtypes = [i]
        L.mgn_status_string.restype = ctypes.c_char_p
        L.mgn_version.argtypes = []
        L.mgn_version.restype = i
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream: Optional[int]) -> Optional[int]:
    if stream is not None:
        return stream
    return torch.cuda.current_stream().cuda_stream


def _dims(q: torch.Tensor):
    B, H, S, D = q.shape
    return int(B), int(H), int(S), int(D)


def mgn_attn_fwd(q, k, v, o, lse, causal: bool, scale: float, mode: int, stream: Optional[int] = None) -> None:
    B, H, S, D = _dims(q)
    st = lib().mgn_attn_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), B, H, S, D,
                            int(causal), float(scale), int(mode), _stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_attn_fwd")


def mgn_attn_bwd_workspace_bytes(B: int, H: int, S: int, D: int, mode: int) -> int:
    return int(lib().mgn_attn_bwd_workspace_bytes(B, H, S, D, mode))


def mgn_attn_bwd(q, k, v, o, d_o, lse, dq, dk, dv, workspace, causal: bool, scale: float, mode: int,
                 stream: Optional[int] = None) -> None:
    B, H, S, D = _dims(q)
    st = lib().mgn_attn_bwd(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(d_o), _ptr(lse), _ptr(dq), _ptr(dk),
                            _ptr(dv), _ptr(workspace), workspace.numel() * workspace.element_size(),
                            B, H, S, D, int(causal), float(scale), int(mode), _stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_attn_bwd")


def _ext_dims(q: torch.Tensor, k: torch.Tensor):
    B, H, Sq, D = q.shape
    _, Hkv, Sk, _ = k.shape
    return int(B), int(H), int(Hkv), int(Sq), int(Sk), int(D)


def mgn_attn_fwd_ext(q, k, v, o, lse, causal: bool, scale: float, mode: int, stream: Optional[int] = None) -> None:
    """q, o: [B,H,Sq,D]; k, v: [B,Hkv,Sk,D] (cross-attention, grouped key/value heads)."""
    B, H, Hkv, Sq, Sk, D = _ext_dims(q, k)
    st = lib().mgn_attn_fwd_ext(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), B, H, Hkv, Sq, Sk, D,
                                int(causal), float(scale), int(mode), _stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_attn_fwd_ext")


def mgn_attn_bwd_ext(q, k, v, o, d_o, lse, dq, dk, dv, workspace, causal: bool, scale: float, mode: int,
                     stream: Optional[int] = None) -> None:
    B, H, Hkv, Sq, Sk, D = _ext_dims(q, k)
    st = lib().mgn_attn_bwd_ext(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(d_o), _ptr(lse), _ptr(dq), _ptr(dk),
                                _ptr(dv), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                B, H, Hkv, Sq, Sk, D, int(causal), float(scale), int(mode), _stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_attn_bwd_ext")


def mgn_attn_fwd_accel_workspace_bytes(B: int, H: int, Hkv: int, Sq: int, Sk: int, D: int) -> int:
    return int(lib().mgn_attn_fwd_accel_workspace_bytes(B, H, Hkv, Sq, Sk, D))


def mgn_attn_fwd_accel(q, k, v, o, lse, workspace, causal: bool, scale: float, stream: Optional[int] = None) -> None:
    """Forward of the accelerated policy: f32 tensors, f16 tensor-core products, f32 O and LSE."""
    B, H, Hkv, Sq, Sk, D = _ext_dims(q, k)
    st = lib().mgn_attn_fwd_accel(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(workspace),
                                  workspace.numel() * workspace.element_size(), B, H, Hkv, Sq, Sk, D,
                                  int(causal), float(scale), _stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_attn_fwd_accel")


def mgn_attn_bwd_deterministic(q, k, v, o, d_o, lse, dq, dk, dv, workspace, causal: bool, scale: float,
                               mode: int, stream: Optional[int] = None) -> None:
    """Backward without floating-point atomics (both modes): bit-identical from run to run."""
    B, H, Hkv, Sq, Sk, D = _ext_dims(q, k)
    st = lib().mgn_attn_bwd_deterministic(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(d_o), _ptr(lse), _ptr(dq),
                                          _ptr(dk), _ptr(dv), _ptr(workspace),
                                          workspace.numel() * workspace.element_size(), B, H, Hkv, Sq, Sk, D,
                                          int(causal), float(scale), int(mode), _stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_attn_bwd_deterministic")


def mgn_attn_bwd_noalloc(q, k, v, o, d_o, lse, dq, dk, dv, causal: bool, scale: float, mode: int,
                         stream: Optional[int] = None) -> None:
    """Backward without a caller workspace: for callers that may not allocate device memory.
    Uses the library's built-in scratch array; sizes beyond it raise MgnError(MGN_ERR_WORKSPACE)."""
    B, H, S, D = _dims(q)
    st = lib().mgn_attn_bwd_noalloc(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(d_o), _ptr(lse), _ptr(dq), _ptr(dk),
                                    _ptr(dv), B, H, S, D, int(causal), float(scale), int(mode), _stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_attn_bwd_noalloc")


def mgn_attn_bwd_noalloc_max_workspace_bytes() -> int:
    return int(lib().mgn_attn_bwd_noalloc_max_workspace_bytes())


def mgn_attn_check(stream: Optional[int] = None) -> None:
    st = lib().mgn_attn_check(_stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_attn_check")


def mgn_attn_profile_events(before_main: Optional[int], after_main: Optional[int]) -> None:
    st = lib().mgn_attn_profile_events(before_main, after_main)
    if st != MGN_OK:
        raise MgnError(st, "mgn_attn_profile_events")


def mgn_attn_fast_item_order(order: int) -> None:
    st = lib().mgn_attn_fast_item_order(int(order))
    if st != MGN_OK:
        raise MgnError(st, "mgn_attn_fast_item_order")


def mgn_attn_strict_tiles(B: int, H: int, H_kv: int, S_q: int, S_k: int, D: int, causal: bool):
    """(fwd_bm, fwd_bn, bwd_bm, bwd_bn): tile shapes the strict kernels run this problem with."""
    out = (ctypes.c_int * 4)()
    st = lib().mgn_attn_strict_tiles(B, H, H_kv, S_q, S_k, D, int(bool(causal)), out)
    if st != MGN_OK:
        raise MgnError(st, "mgn_attn_strict_tiles")
    return tuple(out)


def mgn_measure_fp32_ffma_tflops(stream: Optional[int] = None) -> float:
    scratch = torch.zeros(4, dtype=torch.float32, device="cuda")
    out = ctypes.c_double(0.0)
    st = lib().mgn_measure_fp32_ffma_tflops(_ptr(scratch), ctypes.byref(out), _stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_measure_fp32_ffma_tflops")
    return float(out.value)


def mgn_out_proj_fwd(o, w, y, mode: int, stream: Optional[int] = None) -> None:
    B, H, S, D = _dims(o)
    st = lib().mgn_out_proj_fwd(_ptr(o), _ptr(w), _ptr(y), B, H, S, D, int(w.shape[1]), int(mode), _stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_out_proj_fwd")


def mgn_out_proj_bwd_data(d_y, w, o, d_o, delta, mode: int, stream: Optional[int] = None) -> None:
    B, H, S, D = _dims(o)
    st = lib().mgn_out_proj_bwd_data(_ptr(d_y), _ptr(w), _ptr(o), _ptr(d_o), _ptr(delta), B, H, S, D,
                                     int(w.shape[1]), int(mode), _stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_out_proj_bwd_data")


def mgn_out_proj_bwd_weight(o, d_y, d_w, mode: int, stream: Optional[int] = None) -> None:
    B, H, S, D = _dims(o)
    st = lib().mgn_out_proj_bwd_weight(_ptr(o), _ptr(d_y), _ptr(d_w), B, H, S, D, int(d_w.shape[1]), int(mode), _stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_out_proj_bwd_weight")


def mgn_qkv_rope_fwd(x, w, cos_t, sin_t, q, k, v, mode: int, stream: Optional[int] = None) -> None:
    B, H, S, D = _dims(q)
    st = lib().mgn_qkv_rope_fwd(_ptr(x), _ptr(w), _ptr(cos_t), _ptr(sin_t), _ptr(q), _ptr(k), _ptr(v), B, S,
                                int(x.shape[2]), H, int(k.shape[1]), D, int(mode), _stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_qkv_rope_fwd")


def mgn_rope_bwd_inplace(dq, dk, cos_t, sin_t, mode: int, stream: Optional[int] = None) -> None:
    """dq [B,H,S,D], dk [B,Hkv,S,D] rotated in place by the opposite angles (gradient of the rotary embedding)."""
    B, H, S, D = _dims(dq)
    st = lib().mgn_rope_bwd_inplace(_ptr(dq), _ptr(dk), _ptr(cos_t), _ptr(sin_t), B, H, int(dk.shape[1]), S, D,
                                    int(mode), _stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_rope_bwd_inplace")


def mgn_qkv_bwd_data(gq, gk, gv, w, dx, mode: int, stream: Optional[int] = None) -> None:
    """dx [B,S,E] = (gq | gk | gv heads concatenated) w; gq [B,H,S,D], gk, gv [B,Hkv,S,D], w [(H+2Hkv)D, E]."""
    B, H, S, D = _dims(gq)
    st = lib().mgn_qkv_bwd_data(_ptr(gq), _ptr(gk), _ptr(gv), _ptr(w), _ptr(dx), B, S, int(dx.shape[2]), H,
                                int(gk.shape[1]), D, int(mode), _stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_qkv_bwd_data")


def mgn_qkv_bwd_weight(gq, gk, gv, x, dw, mode: int, stream: Optional[int] = None) -> None:
    """dw [(H+2Hkv)D, E] = (gq | gk | gv heads concatenated)^T x; x [B,S,E]."""
    B, H, S, D = _dims(gq)
    st = lib().mgn_qkv_bwd_weight(_ptr(gq), _ptr(gk), _ptr(gv), _ptr(x), _ptr(dw), B, S, int(x.shape[2]), H,
                                  int(gk.shape[1]), D, int(mode), _stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_qkv_bwd_weight")


def mgn_attn_bwd_given_delta(q, k, v, d_o, lse, delta, dq, dk, dv, workspace, causal: bool, scale: float, mode: int,
                             stream: Optional[int] = None) -> None:
    B, H, Hkv, Sq, Sk, D = _ext_dims(q, k)
    st = lib().mgn_attn_bwd_given_delta(_ptr(q), _ptr(k), _ptr(v), _ptr(d_o), _ptr(lse), _ptr(delta), _ptr(dq),
                                        _ptr(dk), _ptr(dv), _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), B, H, Hkv, Sq, Sk, D,
                                        int(causal), float(scale), int(mode), _stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_attn_bwd_given_delta")


def mgn_selftest_wait_timeout(gave_up: Optional[torch.Tensor] = None, stream: Optional[int] = None) -> None:
    st = lib().mgn_selftest_wait_timeout(_ptr(gave_up), _stream(stream))
    if st != MGN_OK:
        raise MgnError(st, "mgn_selftest_wait_timeout")


def mgn_status_string(status: int) -> str:
    return lib().mgn_status_string(int(status)).decode()


def mgn_version() -> int:
    return int(lib().mgn_version())


def alloc_workspace(B: int, H: int, S: int, D: int, mode: int, device="cuda") -> torch.Tensor:
    """Convenience: a uint8 device buffer of the size mgn_attn_bwd needs (256-byte aligned by torch)."""
    return torch.empty(mgn_attn_bwd_workspace_bytes(B, H, S, D, mode), dtype=torch.uint8, device=device)

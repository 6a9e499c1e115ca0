"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
symbol the header declares, and rejects bad arguments in the documented order."""
import ctypes
import os
import re

import pytest

from paper_2608_01563_b200 import build as mgn_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    mgn_build.build()
    from paper_2608_01563_b200 import binding
    return binding.lib()


def declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(mgn_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(lib):
    syms = declared_symbols()
    assert {"mgn_attn_fwd", "mgn_attn_bwd", "mgn_attn_bwd_workspace_bytes", "mgn_attn_check",
            "mgn_status_string", "mgn_version", "mgn_attn_profile_events", "mgn_attn_bwd_noalloc", "mgn_measure_fp32_ffma_tflops",
            "mgn_attn_fast_item_order", "mgn_attn_fwd_ext", "mgn_attn_bwd_ext",
            "mgn_attn_bwd_deterministic", "mgn_attn_fwd_accel", "mgn_attn_fwd_accel_workspace_bytes",
            "mgn_attn_strict_tiles", "mgn_selftest_wait_timeout", "mgn_out_proj_fwd", "mgn_out_proj_bwd_data",
            "mgn_attn_bwd_given_delta", "mgn_out_proj_bwd_weight", "mgn_qkv_rope_fwd", "mgn_rope_bwd_inplace",
            "mgn_qkv_bwd_data", "mgn_qkv_bwd_weight"} <= set(syms)
    for s in syms:
        assert getattr(lib, s) is not None


def test_item_order_hook_validates_its_argument(lib):
    assert lib.mgn_attn_fast_item_order(2) == 1       # MGN_ERR_INVALID_ARG
    assert lib.mgn_attn_fast_item_order(-2) == 1
    for order in (0, 1, -1):
        assert lib.mgn_attn_fast_item_order(order) == 0


def test_version_and_status_strings(lib):
    assert lib.mgn_version() >= 100
    names = [lib.mgn_status_string(i).decode() for i in range(8)]
    assert names[0] == "MGN_OK" and len(set(names)) == 8
    assert lib.mgn_status_string(99).decode() == "MGN_ERR_UNKNOWN"


def test_workspace_bytes(lib):
    f = lib.mgn_attn_bwd_workspace_bytes
    assert f(8, 12, 1024, 64, 0) >= 8 * 12 * 1024 * 4
    assert f(8, 12, 1024, 64, 1) >= 8 * 12 * 1024 * 4 + 8 * 12 * 1024 * 64 * 4
    assert f(8, 12, 1024, 64, 0) % 256 == 0
    for bad in [(0, 1, 1, 64, 0), (1, 1, 1, 48, 0), (1, 1, 1, 64, 2), (1, -1, 1, 64, 0)]:
        assert f(*bad) == 0


A = 1 << 20  # a fake, 16-byte aligned, never dereferenced device address


def fwd(lib, q=A, k=A, v=A, o=A, lse=A, B=1, H=1, S=8, D=64, causal=0, scale=1.0, mode=0):
    return lib.mgn_attn_fwd(q, k, v, o, lse, B, H, S, D, causal, scale, mode, None)


def bwd(lib, ptrs=None, ws=A, ws_bytes=1 << 30, B=1, H=1, S=8, D=64, causal=0, scale=1.0, mode=0):
    p = [A] * 9 if ptrs is None else ptrs
    return lib.mgn_attn_bwd(*p, ws, ws_bytes, B, H, S, D, causal, scale, mode, None)


def test_forward_argument_validation_order(lib):
    INVALID, UNSUPPORTED, MISALIGNED = 1, 2, 3
    assert fwd(lib, q=None) == INVALID
    assert fwd(lib, lse=None) == INVALID
    assert fwd(lib, S=0) == INVALID
    assert fwd(lib, B=-1) == INVALID
    assert fwd(lib, causal=2) == INVALID
    assert fwd(lib, scale=float("nan")) == INVALID
    assert fwd(lib, scale=float("inf")) == INVALID
    assert fwd(lib, mode=5) == INVALID
    assert fwd(lib, D=48) == UNSUPPORTED
    assert fwd(lib, D=256) == UNSUPPORTED
    assert fwd(lib, B=1 << 20, H=1 << 20) == UNSUPPORTED
    assert fwd(lib, q=A + 4) == MISALIGNED
    assert fwd(lib, o=A + 8) == MISALIGNED
    # invalid beats unsupported beats misaligned
    assert fwd(lib, q=A + 4, D=48) == UNSUPPORTED
    assert fwd(lib, q=A + 4, D=48, S=0) == INVALID
    # a fully valid call gets past validation; without a usable device it must fail, not compute
    import torch
    if not torch.cuda.is_available():
        assert fwd(lib) in (5, 6)


def test_backward_argument_validation_order(lib):
    INVALID, UNSUPPORTED, MISALIGNED, WORKSPACE = 1, 2, 3, 4
    for idx in range(9):
        p = [A] * 9
        p[idx] = None
        assert bwd(lib, ptrs=p) == INVALID
    for idx in range(9):
        p = [A] * 9
        p[idx] = A + 2
        assert bwd(lib, ptrs=p) == MISALIGNED
    assert bwd(lib, D=100) == UNSUPPORTED
    assert bwd(lib, ws=None) == WORKSPACE
    assert bwd(lib, ws_bytes=16) == WORKSPACE
    assert bwd(lib, ws=A + 16) == WORKSPACE
    need = lib.mgn_attn_bwd_workspace_bytes(1, 1, 8, 64, 1)
    assert bwd(lib, ws_bytes=need - 1, mode=1) == WORKSPACE
    assert bwd(lib, ws=None, ptrs=[A + 4] * 9) == MISALIGNED
    assert bwd(lib, ws=None, S=-3) == INVALID


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    from paper_2608_01563_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError):
        binding.mgn_version()


def test_extended_shape_argument_validation(lib):
    """mgn_attn_fwd_ext / mgn_attn_bwd_ext refuse bad head groups and causal S_q > S_k before any launch."""
    INVALID, UNSUPPORTED, MISALIGNED, WORKSPACE = 1, 2, 3, 4
    vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.mgn_attn_fwd_ext.argtypes = [vp] * 5 + [i] * 7 + [f, i, vp]
    lib.mgn_attn_bwd_ext.argtypes = [vp] * 9 + [vp, sz] + [i] * 7 + [f, i, vp]

    def fx(B=1, H=4, Hkv=2, Sq=8, Sk=16, D=64, causal=0, q=A):
        return lib.mgn_attn_fwd_ext(q, A, A, A, A, B, H, Hkv, Sq, Sk, D, causal, 1.0, 0, None)

    def bx(B=1, H=4, Hkv=2, Sq=8, Sk=16, D=64, causal=0, ws=A, ws_bytes=1 << 30):
        return lib.mgn_attn_bwd_ext(*([A] * 9), ws, ws_bytes, B, H, Hkv, Sq, Sk, D, causal, 1.0, 0, None)

    assert fx(H=4, Hkv=3) == INVALID
    assert fx(Hkv=0) == INVALID
    assert fx(Sk=0) == INVALID
    assert fx(Sq=16, Sk=8, causal=1) == UNSUPPORTED
    assert fx(D=48) == UNSUPPORTED
    assert fx(q=A + 4) == MISALIGNED
    assert bx(H=4, Hkv=3) == INVALID
    assert bx(Sq=16, Sk=8, causal=1) == UNSUPPORTED
    lib.mgn_attn_bwd_deterministic.argtypes = lib.mgn_attn_bwd_ext.argtypes
    det = lambda mode=0, H=4, Hkv=2: lib.mgn_attn_bwd_deterministic(*([A] * 9), A, 1 << 30, 1, H, Hkv, 8, 16, 64, 0,
                                                                   1.0, mode, None)
    assert det(mode=7) == INVALID
    assert det(H=4, Hkv=3) == INVALID
    need = lib.mgn_attn_bwd_workspace_bytes(1, 4, 8, 64, 0)       # sized by the query side
    assert bx(ws_bytes=need - 1) == WORKSPACE
    import torch
    if not torch.cuda.is_available():
        assert fx() in (5, 6) and bx() in (5, 6)


def test_accel_forward_argument_validation(lib):
    INVALID, UNSUPPORTED, MISALIGNED, WORKSPACE = 1, 2, 3, 4
    vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.mgn_attn_fwd_accel.argtypes = [vp] * 5 + [vp, sz] + [i] * 7 + [f, vp]
    lib.mgn_attn_fwd_accel_workspace_bytes.argtypes = [i] * 6
    lib.mgn_attn_fwd_accel_workspace_bytes.restype = sz
    need = lib.mgn_attn_fwd_accel_workspace_bytes(1, 4, 2, 8, 16, 64)
    assert need >= (4 * 8 + 2 * 2 * 16) * 64 * 2 and need % 256 == 0
    assert lib.mgn_attn_fwd_accel_workspace_bytes(1, 4, 2, 8, 16, 32) == 0       # the f16 forward takes D in {64,128} only

    def fa(D=64, Hkv=2, ws=A, ws_bytes=1 << 30, q=A):
        return lib.mgn_attn_fwd_accel(q, A, A, A, A, ws, ws_bytes, 1, 4, Hkv, 8, 16, D, 0, 1.0, None)

    assert fa(D=32) == UNSUPPORTED
    assert fa(Hkv=3) == INVALID
    assert fa(q=A + 4) == MISALIGNED
    assert fa(ws=None) == WORKSPACE
    assert fa(ws_bytes=need - 1) == WORKSPACE
    assert fa(ws=A + 16) == WORKSPACE


def test_strict_tile_shapes_follow_the_padded_work():
    """Host-only query: short ragged lengths at D = 64 get the low-padding tiles, everything else the defaults."""
    from paper_2608_01563_b200 import binding
    tiles = binding.mgn_attn_strict_tiles
    assert tiles(32, 12, 12, 197, 197, 64, False) == (40, 112, 40, 64)     # 200 x 224 and 200 x 256 instead of 256 x 256
    assert tiles(1, 4, 4, 197, 197, 64, True) == (40, 112, 40, 64)
    assert tiles(8, 12, 12, 1024, 1024, 64, True) == (64, 128, 64, 64)     # long sequences keep the defaults
    assert tiles(1, 2, 2, 128, 128, 64, False) == (64, 128, 64, 64)        # an exact fit stays
    assert tiles(1, 2, 2, 256, 256, 64, True) == (64, 128, 64, 64)
    assert tiles(1, 2, 2, 197, 197, 128, False) == (64, 64, 32, 64)        # other head sizes have one shape
    assert tiles(1, 2, 2, 64, 64, 32, False) == (64, 128, 64, 64)
    assert tiles(2, 8, 2, 150, 400, 64, True) == (40, 112, 40, 64)         # 150 rows: 160 executed instead of 192
    assert tiles(2, 8, 8, 50, 16, 64, False) == (64, 128, 64, 64)          # one tile either way
    # the chosen shape never executes more padded work than the default
    def work(Sq, Sk, bm, bn, causal):
        n_qt, n_kt = -(-Sq // bm), -(-Sk // bn)
        pairs = 0
        for qt in range(n_qt):
            i_last = min(qt * bm + bm, Sq) - 1
            pairs += min((i_last + Sk - Sq) // bn + 1, n_kt) if causal else n_kt
        return pairs * bm * bn
    for Sq, Sk, causal in [(197, 197, False), (41, 300, True), (300, 300, True), (77, 77, False), (500, 512, True),
                           (50, 16, False), (1, 300, True), (129, 129, False), (513, 513, False)]:
        fbm, fbn, bbm, bbn = tiles(1, 2, 2, Sq, Sk, 64, causal)
        assert work(Sq, Sk, fbm, fbn, causal) <= work(Sq, Sk, 64, 128, causal)
        assert work(Sq, Sk, bbm, bbn, causal) <= work(Sq, Sk, 64, 64, causal)
    with pytest.raises(binding.MgnError):
        tiles(1, 3, 2, 8, 8, 64, False)
    with pytest.raises(binding.MgnError):
        tiles(1, 2, 2, 16, 8, 64, True)
    with pytest.raises(binding.MgnError):
        tiles(1, 2, 2, 8, 8, 48, False)


def test_projection_entry_points_validate_before_any_launch(lib):
    """mgn_out_proj_*, mgn_qkv_rope_fwd and mgn_attn_bwd_given_delta name argument errors in the documented
    order (INVALID_ARG, UNSUPPORTED, MISALIGNED, WORKSPACE) without touching a device."""
    import ctypes
    vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    INVALID, UNSUPPORTED, MISALIGNED, WORKSPACE = 1, 2, 3, 4
    lib.mgn_out_proj_fwd.argtypes = [vp, vp, vp, i, i, i, i, i, i, vp]
    lib.mgn_out_proj_bwd_data.argtypes = [vp] * 5 + [i] * 6 + [vp]
    lib.mgn_out_proj_bwd_weight.argtypes = [vp, vp, vp, i, i, i, i, i, i, vp]
    lib.mgn_qkv_rope_fwd.argtypes = [vp] * 7 + [i] * 7 + [vp]
    lib.mgn_attn_bwd_given_delta.argtypes = [vp] * 9 + [vp, sz] + [i] * 7 + [f, i, vp]

    def pf(o=A, w=A, y=A, B=1, H=2, S=8, D=64, E=64, mode=1):
        return lib.mgn_out_proj_fwd(o, w, y, B, H, S, D, E, mode, None)

    assert pf(o=None) == INVALID and pf(y=None) == INVALID
    assert pf(S=0) == INVALID and pf(E=-8) == INVALID and pf(mode=3) == INVALID
    assert pf(mode=0) == UNSUPPORTED                       # strict-mode projections are not built
    assert pf(D=32) == UNSUPPORTED and pf(D=48) == UNSUPPORTED
    assert pf(E=60) == UNSUPPORTED                         # rows of E elements must be whole 16-byte pieces
    assert pf(w=A + 2) == MISALIGNED
    assert pf(w=A + 2, E=60) == UNSUPPORTED and pf(w=A + 2, E=60, H=0) == INVALID

    def pd(ptrs=None, delta=A, D=64, E=64, mode=1):
        p = [A] * 4 if ptrs is None else ptrs
        return lib.mgn_out_proj_bwd_data(*p, delta, 1, 2, 8, D, E, mode, None)

    for idx in range(4):
        p = [A] * 4
        p[idx] = None
        assert pd(ptrs=p) == INVALID
    assert pd(delta=None) == INVALID and pd(delta=A + 4) == MISALIGNED and pd(D=100) == UNSUPPORTED

    assert lib.mgn_out_proj_bwd_weight(A, A, None, 1, 2, 8, 64, 64, 1, None) == INVALID
    assert lib.mgn_out_proj_bwd_weight(A, A, A, 1, 2, 8, 64, 12, 1, None) == UNSUPPORTED

    def qk(ptrs=None, Hkv=1, D=128, E=64, mode=1):
        p = [A] * 7 if ptrs is None else ptrs
        return lib.mgn_qkv_rope_fwd(*p, 1, 8, E, 2, Hkv, D, mode, None)

    for idx in range(7):
        p = [A] * 7
        p[idx] = None
        assert qk(ptrs=p) == INVALID
    assert qk(Hkv=0) == INVALID and qk(D=32) == UNSUPPORTED and qk(mode=0) == UNSUPPORTED
    p = [A] * 7
    p[3] = A + 8                                            # the sine table
    assert qk(ptrs=p) == MISALIGNED

    # the backward of the QKV projection: opposite rotation in place, data gradient, weight gradient
    lib.mgn_rope_bwd_inplace.argtypes = [vp] * 4 + [i] * 6 + [vp]
    lib.mgn_qkv_bwd_data.argtypes = [vp] * 5 + [i] * 7 + [vp]
    lib.mgn_qkv_bwd_weight.argtypes = [vp] * 5 + [i] * 7 + [vp]

    def rb(ptrs=None, Hkv=1, D=128, mode=1):
        p = [A] * 4 if ptrs is None else ptrs
        return lib.mgn_rope_bwd_inplace(*p, 1, 2, Hkv, 8, D, mode, None)

    for idx in range(4):
        p = [A] * 4
        p[idx] = None
        assert rb(ptrs=p) == INVALID
    assert rb(Hkv=0) == INVALID and rb(D=32) == UNSUPPORTED and rb(mode=0) == UNSUPPORTED and rb(mode=7) == INVALID
    p = [A] * 4
    p[2] = A + 4                                            # the cosine table
    assert rb(ptrs=p) == MISALIGNED

    for fn in (lib.mgn_qkv_bwd_data, lib.mgn_qkv_bwd_weight):
        def qb(ptrs=None, Hkv=1, D=64, E=64, mode=1, S=8):
            p = [A] * 5 if ptrs is None else ptrs
            return fn(*p, 1, S, E, 2, Hkv, D, mode, None)

        for idx in range(5):
            p = [A] * 5
            p[idx] = None
            assert qb(ptrs=p) == INVALID
        assert qb(Hkv=0) == INVALID and qb(S=0) == INVALID and qb(mode=0) == UNSUPPORTED
        assert qb(D=32) == UNSUPPORTED and qb(E=60) == UNSUPPORTED
        p = [A] * 5
        p[2] = A + 2                                        # the value gradient
        assert qb(ptrs=p) == MISALIGNED

    def gd(ptrs=None, ws=A, ws_bytes=1 << 30, Sq=8, Sk=16, D=64, causal=0, mode=0, H=4, Hkv=2):
        p = [A] * 9 if ptrs is None else ptrs
        return lib.mgn_attn_bwd_given_delta(*p, ws, ws_bytes, 1, H, Hkv, Sq, Sk, D, causal, 1.0, mode, None)

    for idx in range(9):                                    # q, k, v, d_o, lse, delta, dq, dk, dv
        p = [A] * 9
        p[idx] = None
        assert gd(ptrs=p) == INVALID
    assert gd(Hkv=3) == INVALID and gd(Sq=32, Sk=16, causal=1) == UNSUPPORTED and gd(D=48) == UNSUPPORTED
    p = [A] * 9
    p[5] = A + 4                                            # delta
    assert gd(ptrs=p) == MISALIGNED
    assert gd(ws=None) == WORKSPACE and gd(ws_bytes=8) == WORKSPACE

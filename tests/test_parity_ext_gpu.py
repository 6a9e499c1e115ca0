"""Cross-attention and grouped key/value heads (mgn_attn_fwd_ext / mgn_attn_bwd_ext): CUDA path vs
the f64 oracle of the same definition, element by element, in both modes.  Shapes follow the
paper's cross-attention workloads (50 action tokens over 16 context tokens; 77-token text context)
and decoder-style grouped heads; lengths span several tiles with ragged tails, and the causal cases
use offsets S_k - S_q that are not multiples of any tile size."""
import math

import pytest
import torch

from paper_2608_01563_b200 import binding as mgn
from paper_2608_01563_b200 import inputs as synth

import helpers as hp

pytestmark = pytest.mark.gpu

CASES = [
    # B, H, Hkv, Sq, Sk, D, causal
    (2, 8, 8, 50, 16, 64, False),        # more queries than keys
    (2, 8, 8, 16, 50, 64, False),
    (1, 8, 2, 33, 77, 64, False),        # text-context length, grouped heads
    (1, 12, 4, 200, 600, 128, False),    # several tiles each way, ragged
    (2, 8, 2, 300, 300, 64, True),       # grouped heads, square causal, ragged
    (1, 6, 1, 257, 257, 128, True),      # multi-query attention
    (1, 4, 2, 100, 260, 64, True),       # bottom-right causal, offset 160
    (1, 4, 4, 257, 520, 128, True),      # offset 263: two masked query blocks per key block
    (1, 4, 1, 1, 300, 64, True),         # a single query row sees every key
    (1, 16, 4, 1, 1, 128, False),
]


def _inputs(seed, B, H, Hkv, Sq, Sk, D, dtype):
    q, _, _, d_o = synth.random_inputs(seed, B, H, Sq, D, dtype=dtype)
    _, k, v, _ = synth.random_inputs(seed + 1, B, Hkv, Sk, D, dtype=dtype)
    return q, k, v, d_o


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal", CASES)
def test_strict_matches_oracle(B, H, Hkv, Sq, Sk, D, causal):
    scale = 1.0 / math.sqrt(D)
    q, k, v, d_o = _inputs(300, B, H, Hkv, Sq, Sk, D, torch.float32)
    got = hp.run_cuda_ext(q, k, v, d_o, causal, scale, mgn.MODE_STRICT_F32)
    ref = hp.run_oracle_ext(q, k, v, d_o, causal, scale)
    hp.check_strict(got, ref, literal_max_abs=False, label=f"ext strict {B,H,Hkv,Sq,Sk,D,causal} ")


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal", CASES)
def test_fast_matches_oracle(B, H, Hkv, Sq, Sk, D, causal):
    scale = 1.0 / math.sqrt(D)
    q, k, v, d_o = _inputs(400, B, H, Hkv, Sq, Sk, D, torch.bfloat16)
    got = hp.run_cuda_ext(q, k, v, d_o, causal, scale, mgn.MODE_FAST_BF16)
    ref = hp.run_oracle_ext(q, k, v, d_o, causal, scale)
    hp.check_fast(got, ref, label=f"ext fast {B,H,Hkv,Sq,Sk,D,causal} ")


@pytest.mark.parametrize("order", [0, 1])
def test_fast_grouped_decoder_shape_in_both_item_orders(order):
    """Grouped heads at a decoder-like size (several items per CTA): B=2, H=32, H_kv=8, S=1024, D=128."""
    B, H, Hkv, S, D = 2, 32, 8, 1024, 128
    scale = 1.0 / math.sqrt(D)
    q, k, v, d_o = _inputs(500 + order, B, H, Hkv, S, S, D, torch.bfloat16)
    mgn.mgn_attn_fast_item_order(order)
    try:
        got = hp.run_cuda_ext(q, k, v, d_o, True, scale, mgn.MODE_FAST_BF16)
    finally:
        mgn.mgn_attn_fast_item_order(-1)
    ref = hp.run_oracle_ext(q, k, v, d_o, True, scale)
    hp.check_fast(got, ref, label=f"ext fast grouped order={order} ")


def test_strict_grouped_decoder_shape():
    B, H, Hkv, S, D = 1, 16, 4, 1024, 64
    scale = 1.0 / math.sqrt(D)
    q, k, v, d_o = _inputs(600, B, H, Hkv, S, S, D, torch.float32)
    got = hp.run_cuda_ext(q, k, v, d_o, True, scale, mgn.MODE_STRICT_F32)
    ref = hp.run_oracle_ext(q, k, v, d_o, True, scale)
    hp.check_strict(got, ref, literal_max_abs=False, label="ext strict grouped ")


def test_argument_errors():
    q = torch.zeros(1, 4, 8, 64, device="cuda")
    k = torch.zeros(1, 3, 8, 64, device="cuda")
    o = torch.empty_like(q)
    lse = torch.empty(1, 4, 8, device="cuda")
    with pytest.raises(mgn.MgnError) as e:
        mgn.mgn_attn_fwd_ext(q, k, k, o, lse, False, 1.0, mgn.MODE_STRICT_F32)     # 4 % 3 != 0
    assert e.value.status == 1
    k2 = torch.zeros(1, 4, 4, 64, device="cuda")
    with pytest.raises(mgn.MgnError) as e:
        mgn.mgn_attn_fwd_ext(q, k2, k2, o, lse, True, 1.0, mgn.MODE_STRICT_F32)    # causal with S_q > S_k
    assert e.value.status == 2


def _group_slice(w, t_q, t_k, b, hk):
    """Tensors of one (batch, key/value head) group: its G query heads and its one K/V head."""
    G = w.H // w.Hkv
    return t_q[b:b + 1, hk * G:(hk + 1) * G], t_k[b:b + 1, hk:hk + 1]


@pytest.mark.parametrize("name", ["gqa_decoder", "cross_attn_text", "cross_attn_action", "gqa_suffix"])
@pytest.mark.parametrize("mode", [mgn.MODE_STRICT_F32, mgn.MODE_FAST_BF16])
def test_measured_workloads_on_sampled_groups(name, mode):
    """The workloads the benchmark times, at full size on the GPU; the oracle checks two
    (batch, key/value head) groups -- a group is closed under the dk, dv sums."""
    w = synth.EXT_WORKLOADS[name]
    dt = torch.float32 if mode == mgn.MODE_STRICT_F32 else torch.bfloat16
    q, k, v, d_o = synth.make_inputs_ext(w, dtype=dt)
    got = hp.run_cuda_ext(q, k, v, d_o, w.causal, w.scale, mode)
    G = w.H // w.Hkv
    for b, hk in ((0, 0), (w.B - 1, w.Hkv - 1)):
        qs, ks = _group_slice(w, q, k, b, hk)
        dos, vs = _group_slice(w, d_o, v, b, hk)
        ref = hp.run_oracle_ext(qs, ks, vs, dos, w.causal, w.scale)
        sub = {"O": got["O"][b:b + 1, hk * G:(hk + 1) * G], "LSE": got["LSE"][b:b + 1, hk * G:(hk + 1) * G],
               "dQ": got["dQ"][b:b + 1, hk * G:(hk + 1) * G], "dK": got["dK"][b:b + 1, hk:hk + 1],
               "dV": got["dV"][b:b + 1, hk:hk + 1]}
        if mode == mgn.MODE_STRICT_F32:
            hp.check_strict(sub, ref, literal_max_abs=False, label=f"{name} strict group {b,hk} ")
        else:
            hp.check_fast(sub, ref, label=f"{name} fast group {b,hk} ")

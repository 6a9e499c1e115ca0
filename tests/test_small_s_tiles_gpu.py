"""Short ragged sequences in strict mode: the kernels switch to tiles with less padding (40-row
query tiles, 112-key forward tiles) when that cuts the executed work by more than an eighth.  Every
shape here is checked to select those tiles (mgn_attn_strict_tiles) and then compared with the f64
oracle element by element: ragged tails in both directions, causal masks with and without an
offset, grouped key/value heads, and the deterministic backward."""
import math

import pytest
import torch

from paper_2608_01563_b200 import binding as mgn
from paper_2608_01563_b200 import inputs as synth

import helpers as hp

pytestmark = pytest.mark.gpu

CASES = [
    # B, H, Hkv, Sq, Sk, D, causal
    (3, 4, 4, 197, 197, 64, False),      # the vision-transformer length
    (2, 4, 4, 197, 197, 64, True),
    (1, 8, 2, 150, 400, 64, True),       # bottom-right causal, offset 250, grouped heads
    (2, 6, 6, 129, 129, 64, False),      # one row past a 64-row tile
    (1, 8, 2, 33, 77, 64, False),        # text-context cross-attention
    (1, 4, 1, 81, 225, 64, True),        # one row into the third query tile, one key into the third key tile
]


def _inputs(seed, B, H, Hkv, Sq, Sk, D):
    q, _, _, d_o = synth.random_inputs(seed, B, H, Sq, D, dtype=torch.float32)
    _, k, v, _ = synth.random_inputs(seed + 1, B, Hkv, Sk, D, dtype=torch.float32)
    return q, k, v, d_o


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal", CASES)
def test_low_padding_tiles_match_the_oracle(B, H, Hkv, Sq, Sk, D, causal):
    fbm, fbn, bbm, bbn = mgn.mgn_attn_strict_tiles(B, H, Hkv, Sq, Sk, D, causal)
    assert (fbm, fbn) == (40, 112) or bbm == 40, "this shape was meant to select the alternative tiles"
    scale = 1.0 / math.sqrt(D)
    q, k, v, d_o = _inputs(900, B, H, Hkv, Sq, Sk, D)
    got = hp.run_cuda_ext(q, k, v, d_o, causal, scale, mgn.MODE_STRICT_F32)
    ref = hp.run_oracle_ext(q, k, v, d_o, causal, scale)
    hp.check_strict(got, ref, literal_max_abs=False, label=f"small-S tiles {B,H,Hkv,Sq,Sk,D,causal} ")


def test_square_entry_point_uses_them_too():
    """mgn_attn_fwd / mgn_attn_bwd (square multi-head build of the kernels) on the ViT length."""
    w = synth.WORKLOADS["vit_b_ragged"]
    assert mgn.mgn_attn_strict_tiles(w.B, w.H, w.H, w.S, w.S, w.D, w.causal) == (40, 112, 40, 64)
    q, k, v, d_o = synth.random_inputs(901, 2, 3, w.S, w.D, dtype=torch.float32)
    got = hp.select(hp.run_cuda(q, k, v, d_o, True, w.scale, mgn.MODE_STRICT_F32), 2, 3)
    ref = hp.run_oracle(q, k, v, d_o, True, w.scale)
    hp.check_strict(got, ref, literal_max_abs=False, label="small-S tiles square causal ")


# Shapes whose last key tile holds visible keys in its first half only: the forward then runs both
# products of that tile over half of it.  Each keeps the default tiles (checked), so the path taken
# is the half-tile one of the 64 x 128 (D <= 64) and 64 x 64 (D = 128) builds.
HALF_TILE_CASES = [
    # B, H, Hkv, Sq, Sk, D, causal
    (1, 3, 3, 1024, 1024, 64, True),     # every other query tile ends on a half-visible key tile
    (2, 4, 2, 700, 1070, 64, False),     # ragged tail: 46 keys in the ninth key tile
    (1, 4, 4, 600, 650, 64, True),       # bottom-right offset 50: half tiles from the offset and the tail
    (2, 2, 2, 640, 640, 32, True),       # head size 32 (eight-key unrolled groups)
    (1, 4, 1, 600, 592, 128, False),     # D = 128: 16 keys in the tenth 64-key tile
    (1, 2, 2, 540, 550, 128, True),      # D = 128, offset 10
]


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal", HALF_TILE_CASES)
def test_half_visible_key_tiles_match_the_oracle(B, H, Hkv, Sq, Sk, D, causal):
    fbm, fbn, _, _ = mgn.mgn_attn_strict_tiles(B, H, Hkv, Sq, Sk, D, causal)
    assert (fbm, fbn) == ((64, 64) if D == 128 else (64, 128))
    scale = 1.0 / math.sqrt(D)
    q, k, v, d_o = _inputs(950, B, H, Hkv, Sq, Sk, D)
    got = hp.run_cuda_ext(q, k, v, d_o, causal, scale, mgn.MODE_STRICT_F32, run_bwd=False)
    ref = hp.run_oracle_ext(q, k, v, d_o, causal, scale)
    hp.check_strict(got, ref, names=("O", "LSE"), literal_max_abs=False,
                    label=f"half key tiles {B,H,Hkv,Sq,Sk,D,causal} ")

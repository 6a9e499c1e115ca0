"""Fast-mode forward on short key sequences (at most two 128-key blocks): these problems take the
latency path (one small CTA per query tile, one thread per row, classic online softmax).  Element by
element against the f64 oracle through the C ABI, at the fast mode's tolerance."""
import math

import numpy as np
import pytest
import torch

from paper_2608_01563_b200 import binding as mgn
from paper_2608_01563_b200 import inputs as synth

import helpers as hp

pytestmark = pytest.mark.gpu
MODE = mgn.MODE_FAST_BF16
BF = torch.bfloat16


def _forward(q, k, v, causal, scale):
    B, H, Sq, D = q.shape
    o = hp.Guarded((B, H, Sq, D), BF)
    lse = hp.Guarded((B, H, Sq), torch.float32)
    mgn.mgn_attn_fwd_ext(q.cuda(), k.cuda(), v.cuda(), o.view, lse.view, causal, scale, MODE)
    mgn.mgn_attn_check()
    return o.check("O").double().numpy(), lse.check("LSE").double().numpy()


@pytest.mark.parametrize("B,H,Hkv,Sq,Sk,D,causal", [
    (2, 4, 4, 1000, 77, 64, False),      # many query tiles over one partly filled key block
    (3, 8, 2, 50, 16, 64, False),        # a single 16-key step, grouped heads
    (1, 4, 4, 256, 256, 128, True),      # two blocks, causal: the first query tile sees one block only
    (2, 2, 1, 100, 250, 128, True),      # bottom-right causal offset 150 into the second block
    (1, 3, 3, 300, 129, 64, False),      # one key in the second block
    (2, 6, 3, 197, 197, 32, True),       # head size 32 (zero-padded), ragged both ways
])
def test_short_key_sequences_match_the_oracle(B, H, Hkv, Sq, Sk, D, causal):
    g = torch.Generator().manual_seed(70 + Sq + Sk)
    q = torch.randn(B, H, Sq, D, generator=g).to(BF)
    k = torch.randn(B, Hkv, Sk, D, generator=g).to(BF)
    v = torch.randn(B, Hkv, Sk, D, generator=g).to(BF)
    scale = 1.0 / math.sqrt(D)
    o, lse = _forward(q, k, v, causal, scale)
    ref = hp.run_oracle_ext(q, k, v, torch.zeros_like(q), causal, scale)
    assert hp.rel_l2(o, ref["O"]) <= hp.FAST_REL_L2
    assert hp.rel_l2(lse, ref["LSE"]) <= 1e-3


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("causal", [False, True])
def test_second_block_raises_every_row_maximum(D, causal):
    """Keys of the second block are far larger than those of the first, so every row moves its running
    maximum there and rescales the output it has accumulated (by 2^-40 and less)."""
    B, H, S = 1, 3, 256
    q, k, v, _ = synth.random_inputs(81 + D, B, H, S, D, dtype=torch.float32)
    q[..., 0] = 3.0
    k[:, :, 128:, 0] = 12.0                      # scores of the second block: + 36 * scale * ... over the first
    q, k, v = q.to(BF), k.to(BF), v.to(BF)
    o, lse = _forward(q, k, v, causal, 1.0)
    ref = hp.run_oracle(q, k, v, torch.zeros_like(q), causal, 1.0)
    assert hp.rel_l2(o, ref["O"].reshape(o.shape)) <= hp.FAST_REL_L2
    err = np.abs(lse - ref["LSE"].reshape(lse.shape))
    assert (err <= 2e-2 + 1e-3 * np.abs(ref["LSE"].reshape(lse.shape))).all()

"""The bounded device waits: a wait that runs out must leave the kernel, flag the per-device status
word, make later attention kernels skip their work, and be reported (and cleared) by
mgn_attn_check -- without a hang, a trap or a fault.  The wait is made to run out by the
library's own self-test kernel (1024 polls on a barrier that nothing arrives on)."""
import pytest
import torch

from paper_2608_01563_b200 import binding as mgn
from paper_2608_01563_b200 import inputs as synth

pytestmark = pytest.mark.gpu


def _forward(mode, dtype):
    B, H, S, D = 1, 2, 200, 64
    q, k, v, _ = (t.cuda() for t in synth.random_inputs(21, B, H, S, D, dtype=dtype))
    o = torch.full_like(q, float("nan"))
    lse = torch.full((B, H, S), float("nan"), device="cuda")
    mgn.mgn_attn_fwd(q, k, v, o, lse, True, 0.125, mode)      # returns MGN_OK: it only enqueues
    torch.cuda.synchronize()
    return o, lse


@pytest.mark.parametrize("mode,dtype", [(mgn.MODE_STRICT_F32, torch.float32), (mgn.MODE_FAST_BF16, torch.bfloat16)])
def test_a_wait_that_runs_out_is_reported_once_and_later_kernels_skip_their_work(mode, dtype):
    mgn.mgn_attn_check()                                       # clean state
    gave_up = torch.zeros(1, dtype=torch.int32, device="cuda")
    mgn.mgn_selftest_wait_timeout(gave_up)
    torch.cuda.synchronize()                                   # the kernel returned: nothing hangs
    assert int(gave_up.item()) == 1

    # the device is now flagged: an attention kernel leaves its outputs unwritten
    o, lse = _forward(mode, dtype)
    assert torch.isnan(o.float()).all() and torch.isnan(lse).all()

    with pytest.raises(mgn.MgnError) as e:
        mgn.mgn_attn_check()
    assert e.value.status == 7                                 # MGN_ERR_DEVICE_TIMEOUT, once
    mgn.mgn_attn_check()                                       # cleared: MGN_OK

    # and the library works again
    o, lse = _forward(mode, dtype)
    assert not torch.isnan(o.float()).any() and not torch.isnan(lse).any()
    mgn.mgn_attn_check()

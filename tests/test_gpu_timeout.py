"""A bounded device-side wait that really runs out, in the safe form: nothing hangs, traps or faults.

The dense streaming kernel's last CTAs wait (bounded) for the arrival counter before they turn the partial sums
into the output: each waits until the count reaches the next multiple of the grid size.  The counter is seeded
with grid size - 1, so the launch's arrivals straddle a multiple: all but one finaliser wait for a count this
launch never reaches, and with the budget cut to half a millisecond they give up.  (A one-token launch counts
its arrivals in the accumulator words themselves; the same call makes those words wait for one arrival more than
the launch has.)  Every CTA has streamed its share, added its sums and exits normally; the finalisers that gave
up flag MOE_ERR_TIMEOUT.
Checked: moe_check reports the time-out, clears it and re-arms the ctx's state (arrival counter, accumulators),
and the next ordinary call is bit-identical to a fresh ctx's and matches the CPU checker."""
import numpy as np
import pytest
import torch

from synth import workloads as W
from tests import gpu_util as U

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("sh,T", [(W.TINY, 1), (W.WEARABLE, 1), (W.TINY, 8)])
def test_expired_finaliser_wait_is_reported_and_the_ctx_recovers(sh, T):
    from paper_2503_00245_b200 import binding as B
    lay, t, host = U.build(sh, T, path=B.MOE_PATH_STREAM)
    x = t["x"]
    ref = lay.forward(x).clone()
    torch.cuda.synchronize()
    assert lay.check() == 0
    B.moe_set_finaliser_wait(lay.ctx, 1_000_000)
    B.moe_seed_arrival_counter(lay.ctx, B.moe_device_sm_count() - 1)
    lay.forward(x)                      # output of this call is undefined
    torch.cuda.synchronize()
    assert lay.check() == 5             # MOE_ERR_TIMEOUT, and the state is cleared
    assert lay.check() == 0             # reported once
    B.moe_set_finaliser_wait(lay.ctx, 0)
    for _ in range(3):                  # the re-armed ctx behaves like a fresh one
        y = lay.forward(x).clone()
        torch.cuda.synchronize()
        assert lay.check() == 0
        assert torch.equal(y, ref)
    rel, _, _ = U.check_layer(lay, t, host, sh.top_k)
    assert rel <= U.Y_TOL
    with pytest.raises(B.MoeError):
        B.moe_set_finaliser_wait(lay.ctx, -1)
    lay.close()

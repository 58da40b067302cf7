"""The device-side timeout contract: a bounded wait that runs out makes the kernel record WCC_ERR_TIMEOUT and return
normally; wcc_last_status reports it once, clears it, and the library keeps working.  The wait is made to run out by
waiting on a barrier that nothing arrives on, with the poll limit lowered so that it takes about a millisecond; no
kernel traps, faults or spins without bound."""
import numpy as np
import pytest
import torch

import oracle
from paper_2205_12268_b200 import inputs

pytestmark = pytest.mark.gpu

WCC_ERR_TIMEOUT = 9


@pytest.fixture(scope="module")
def wcc():
    from paper_2205_12268_b200 import build, wcc as w
    build.build()
    assert torch.cuda.is_available()
    w.lib()
    return w


def test_wait_that_runs_out_is_reported_once_and_the_library_keeps_working(wcc):
    assert wcc.last_status() == 0
    wcc.debug_set_wait_limit(1000)
    try:
        wcc.debug_wait_selftest()
        assert wcc.last_status() == WCC_ERR_TIMEOUT
        assert wcc.last_status() == 0                      # reading cleared it
    finally:
        wcc.debug_set_wait_limit(0)                        # back to the default
    w = inputs.custom("after_timeout", 4, 2, 24, 40, 32, 64, "bf16", 3, 0.25, 8, n_sin=4, fmax=3.0)
    x = torch.from_numpy(w.x.view(np.int16)).cuda().view(torch.bfloat16)
    y = wcc.forward(x, torch.from_numpy(w.Wt).cuda(), w.levels, w.k, w.bits)
    assert wcc.last_status() == 0
    want = oracle.forward(w.x_f32(), w.Wt, w.levels, w.k, w.bits, out_bf16=True)
    assert np.array_equal(y.float().cpu().numpy().view(np.uint32), want.view(np.uint32))

"""The scratch-free select entry point (wcc_select_topk_static) against the ordinary one, through the C ABI.

Collected last on purpose (file name): a run that stops at the first failure has then already run everything else.
The entry point serves callers that may not allocate device memory; it must give the same index list and threshold
as wcc_select_topk, call after call, although all calls share one built-in scratch array that keeps old contents."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def wcc():
    from paper_2205_12268_b200 import build, wcc as w
    build.build()
    assert torch.cuda.is_available()
    w.lib()
    return w


def _both(wcc, nrm, k):
    N, P = nrm.shape
    idx = torch.empty((N, k), dtype=torch.int32, device="cuda")
    tau = torch.empty((N,), dtype=torch.float32, device="cuda")
    wcc.select_topk_static(nrm, k, idx, tau)
    ref_idx, ref_tau = wcc.select_topk(nrm, k)
    torch.cuda.synchronize()
    assert wcc.last_status() == 0
    assert torch.equal(idx, ref_idx)                 # integer result: identical
    assert torch.equal(tau, ref_tau)                 # a value copied out of the input: identical


def test_static_scratch_select_matches_on_two_calls_in_a_row(wcc):
    g = torch.Generator(device="cuda").manual_seed(1)
    a = torch.rand((4, 32768), device="cuda", generator=g) ** 3
    _both(wcc, a, 16384)
    # second call right after, other shape and k: nothing of the first call's histograms or counts may leak in
    b = torch.randint(0, 5, (3, 5000), device="cuda", generator=g).float()       # heavy ties
    _both(wcc, b, 1234)
    _both(wcc, a, 1)


def test_static_scratch_select_rejects_what_does_not_fit(wcc):
    assert wcc.lib().wcc_select_workspace_bytes(32, 4096) > wcc.STATIC_SCRATCH_BYTES
    nrm = torch.zeros((32, 4096), device="cuda")
    idx = torch.empty((32, 8), dtype=torch.int32, device="cuda")
    tau = torch.empty((32,), dtype=torch.float32, device="cuda")
    with pytest.raises(wcc.WccError) as e:
        wcc.select_topk_static(nrm, 8, idx, tau)
    assert e.value.code == 7
    with pytest.raises(wcc.WccError) as e:
        wcc.select_topk_static(nrm[:2], 5000, idx, tau)
    assert e.value.code == 3

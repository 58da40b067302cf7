"""The scratch-free select entry point (wcc_select_topk_static) through the C ABI, against the ordinary entry point
and against the CPU oracle.

Collected last on purpose (file name): a run that stops at the first failure has then already run everything else.
The entry point serves callers that may not allocate device memory; it must give the same index list and threshold
as wcc_select_topk, call after call, although all calls share one built-in scratch array that keeps old contents.
Images of up to 131072 positions are selected inside one thread-block cluster and never touch the scratch array (those
cases only exercise the address lookup and the size check); larger images go through the kernels that keep their
histograms, barrier counters, per-image state and chunk counts in it, so the cases that prove anything about stale
scratch contents use 150000 to 200000 positions per image."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def wcc():
    from paper_2205_12268_b200 import build, wcc as w
    build.build()
    assert torch.cuda.is_available()
    w.lib()
    return w


def _check(wcc, nrm, k):
    """static entry point == ordinary entry point == oracle (index lists identical, thresholds identical)."""
    N, P = nrm.shape
    assert wcc.lib().wcc_select_workspace_bytes(N, P) <= wcc.STATIC_SCRATCH_BYTES
    idx = torch.full((N, k), -7, dtype=torch.int32, device="cuda")
    tau = torch.full((N,), float("nan"), dtype=torch.float32, device="cuda")
    wcc.select_topk_static(nrm, k, idx, tau)
    ref_idx, ref_tau = wcc.select_topk(nrm, k)
    torch.cuda.synchronize()
    assert wcc.last_status() == 0
    assert torch.equal(idx, ref_idx)                 # integer result: identical
    assert torch.equal(tau, ref_tau)                 # a value copied out of the input: identical
    want_idx, want_tau = oracle.select_topk(nrm.cpu().numpy(), k)
    assert np.array_equal(idx.cpu().numpy(), want_idx)
    assert np.array_equal(tau.cpu().numpy().view(np.uint32), want_tau.view(np.uint32))


def test_static_scratch_select_small_images_two_calls_in_a_row(wcc):
    g = torch.Generator(device="cuda").manual_seed(1)
    a = torch.rand((4, 32768), device="cuda", generator=g) ** 3
    _check(wcc, a, 16384)
    b = torch.randint(0, 5, (3, 5000), device="cuda", generator=g).float()       # heavy ties
    _check(wcc, b, 1234)
    _check(wcc, a, 1)


def test_static_scratch_select_large_images_reuse_the_scratch_array(wcc):
    """Images beyond one cluster: the histograms, barrier counters, state words and chunk counts live in the built-in
    array.  Calls of different shapes, tie patterns and k follow one another, so each starts from what the previous
    one left behind; every one must still match the ordinary entry point and the oracle."""
    g = torch.Generator(device="cuda").manual_seed(2)
    a = torch.rand((2, 200000), device="cuda", generator=g) ** 2
    a[:, 1000:60000] = 0.25                                                       # a long run of equal norms
    _check(wcc, a, 50000)                                                         # the threshold cuts through the run
    b = torch.randint(0, 7, (13, 150000), device="cuda", generator=g).float()     # more images: more resident blocks
    _check(wcc, b, 77777)
    _check(wcc, a, 3)                                                             # first shape again, other k
    c = torch.rand((3, 180224), device="cuda", generator=g)
    _check(wcc, c, 180224)                                                        # keep everything
    _check(wcc, b[:5].contiguous(), 1)


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

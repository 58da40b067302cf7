"""Maps with large regions of exact zeros (what a ReLU leaves behind): positions whose norm is zero are left out of the
selection's histograms on the GPU, and the threshold may itself be zero.  Everything must still equal the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2205_12268_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def wcc():
    from paper_2205_12268_b200 import build, wcc as w
    build.build()
    assert torch.cuda.is_available()
    w.lib()
    return w


def _sparse(seed, N, Cin, Cout, H, W, dtype, L, gamma, frac_zero_blocks):
    w = inputs.custom("sparse", seed, N, Cin, Cout, H, W, dtype, L, gamma, 8, n_sin=4, fmax=3.0)
    rng = np.random.default_rng(seed)
    blk = 1 << L
    mask = rng.random((N, 1, H // blk, W // blk)) < frac_zero_blocks          # whole transform blocks, all channels
    mask = np.repeat(np.repeat(mask, blk, axis=2), blk, axis=3)
    w.x[np.broadcast_to(mask, w.x.shape)] = 0
    return w


@pytest.mark.parametrize("staged", [False, True], ids=["fused", "staged"])
@pytest.mark.parametrize("cfg", [(2, 12, 20, 32, 64, "f32", 2, 0.7), (2, 40, 24, 64, 64, "bf16", 3, 0.7),
                                  (1, 8, 8, 32, 128, "f32", 1, 0.5)], ids=lambda c: "N%d_%dto%d_%dx%d_%s_L%d_zero%s" % c)
def test_mostly_zero_maps_with_taps(wcc, cfg, staged):
    N, Cin, Cout, H, W, dtype, L, fz = cfg
    for gamma in (0.05, 0.29, 0.31, 0.9):            # fewer / about as many / more kept positions than non-zero norms
        w = _sparse(31, N, Cin, Cout, H, W, dtype, L, gamma, fz)
        x = torch.from_numpy(w.x.view(np.int16)).cuda().view(torch.bfloat16) if dtype == "bf16" else torch.from_numpy(w.x).cuda()
        y, t = wcc.forward(x, torch.from_numpy(w.Wt).cuda(), L, w.k, 8, taps=True, staged=staged)
        assert wcc.last_status() == 0
        want, o = oracle.forward(w.x_f32(), w.Wt, L, w.k, 8, out_bf16=(dtype == "bf16"), taps=True)
        assert (o["nrm2"] == 0).mean() > 0.4
        assert np.array_equal(t["idx"].cpu().numpy(), o["idx"])
        assert np.array_equal(t["acc"].cpu().numpy(), o["acc"].reshape(-1, Cout))
        assert np.array_equal(y.float().cpu().numpy().view(np.uint32), want.view(np.uint32))
        y2 = wcc.forward(x, torch.from_numpy(w.Wt).cuda(), L, w.k, 8, staged=staged)      # threshold-only path
        assert torch.equal(y, y2)


def test_relu_output_as_next_input_is_fast_path_correct(wcc):
    """A zero threshold with ties kept in part takes the threshold-only path (no rank map): same output."""
    w = _sparse(32, 2, 16, 16, 64, 128, "bf16", 3, 0.6, 0.8)
    x = torch.from_numpy(w.x.view(np.int16)).cuda().view(torch.bfloat16)
    Wt = torch.from_numpy(w.Wt).cuda()
    nz = int((oracle.forward(w.x_f32(), w.Wt, 3, w.k, 8, taps=True)[1]["nrm2"] != 0).sum(axis=1).min())
    assert w.k > nz                                   # more positions kept than there are non-zero norms
    y = wcc.forward(x, Wt, 3, w.k, 8, relu=True)
    want = oracle.forward(w.x_f32(), w.Wt, 3, w.k, 8, out_bf16=True, relu=True)
    assert wcc.last_status() == 0
    assert np.array_equal(y.float().cpu().numpy().view(np.uint32), want.view(np.uint32))

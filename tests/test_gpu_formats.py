"""GPU parity of the kept set as a bitmap (wcc_select_topk_bitmap) and of the layer on maps whose sides are no multiples
of 2^levels (wcc_forward_padded), against the oracle."""
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


@pytest.mark.parametrize("shape", [(3, 1000, 250), (2, 4096, 1), (1, 33, 33), (2, 32768, 8192), (1, 200000, 60000)])
def test_bitmap_equals_the_oracles_index_list(wcc, shape):
    N, P, k = shape
    g = torch.Generator(device="cuda").manual_seed(P)
    nrm = torch.rand((N, P), device="cuda", generator=g) ** 2
    nrm[:, : P // 3] = torch.round(nrm[:, : P // 3] * 4) / 4                 # ties
    bm, tau = wcc.select_topk_bitmap(nrm, k)
    assert wcc.last_status() == 0
    idx, tau_o = oracle.select_topk(nrm.cpu().numpy(), k)
    want = oracle.bitmap_of(idx, P)
    assert np.array_equal(bm.cpu().numpy().view(np.uint32), want)
    assert np.array_equal(tau.cpu().numpy().view(np.uint32), tau_o.view(np.uint32))


PADDED = [  # N, Cin, Cout, H, W, dtype, levels, gamma, bits
    (2, 5, 7, 13, 27, "f32", 3, 0.3, 8),
    (1, 24, 40, 33, 65, "bf16", 3, 0.25, 8),          # the shape of a 513 x 1025 map, scaled down
    (2, 8, 8, 10, 14, "f32", 1, 0.5, 8),              # padded width 14: rows the TMA path cannot take
    (1, 6, 6, 30, 50, "bf16", 2, 1.0, 0),
    (1, 12, 20, 32, 64, "f32", 3, 0.4, 8),            # nothing to pad
]


@pytest.mark.parametrize("cfg", PADDED, ids=lambda c: "N%d_%dto%d_%dx%d_%s_L%d_g%s_b%d" % c)
def test_padded_layer(wcc, cfg):
    N, Cin, Cout, H, W, dtype, L, gamma, bits = cfg
    rng = np.random.default_rng(H * W)
    x = (np.maximum(rng.standard_normal((N, Cin, H, W)), 0) + 0.05 * rng.standard_normal((N, Cin, H, W))).astype(np.float32)
    Wt = inputs.weights(3, Cout, Cin)
    unit = 1 << L
    Pp = (-(-H // unit) * unit) * (-(-W // unit) * unit)
    k = inputs.keep_count(gamma, Pp)
    if dtype == "bf16":
        b = inputs.f32_to_bf16_bits(x)
        xd, xh = torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16), inputs.bf16_bits_to_f32(b)
    else:
        xd, xh = torch.from_numpy(x).cuda(), x
    y = wcc.forward_padded(xd, torch.from_numpy(Wt).cuda(), L, k, bits)
    assert wcc.last_status() == 0
    want = oracle.forward_padded(xh, Wt, L, k, bits, out_bf16=(dtype == "bf16"))
    got = y.float().cpu().numpy()
    assert got.shape == want.shape
    if bits:
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    else:
        assert np.abs(got - want).max() <= 2e-2 * np.abs(want).max()

"""GPU parity of the generic wavelet entry points (App. F: WCC with other wavelets) against the oracle: coefficients
and norms bit for bit, the layer's kept indices, codes and accumulators identical, its output within the float tolerance."""
import numpy as np
import pytest
import torch

import oracle
from paper_2205_12268_b200 import inputs, wavelets

pytestmark = pytest.mark.gpu

BANKS = ["haar", "db2", "db3", "db4", "bior2.2"]


@pytest.fixture(scope="module")
def wcc():
    from paper_2205_12268_b200 import build, wcc as w
    build.build()
    assert torch.cuda.is_available()
    w.lib()
    return w


def _bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


@pytest.mark.parametrize("name", BANKS)
@pytest.mark.parametrize("shape", [(2, 3, 16, 24, 1), (1, 5, 32, 64, 3), (2, 2, 8, 8, 2), (1, 4, 64, 96, 2)])
def test_dwt_fwd_inv_bit_exact(wcc, name, shape):
    N, Cc, H, W, L = shape
    dl, dh, rl, rh = wavelets.filter_bank(name)
    x = inputs.feature_map(14, N, Cc, H, W, 4, 3.0).astype(np.float32)
    coef, nrm2 = wcc.dwt_fwd(torch.from_numpy(x).cuda(), L, dl, dh)
    assert wcc.last_status() == 0
    want = oracle.dwt(x, L, dl, dh)
    assert np.array_equal(_bits(coef.cpu().numpy()), _bits(want))
    assert np.array_equal(_bits(nrm2.cpu().numpy()), _bits(oracle.norms(want)))
    back = wcc.dwt_inv(coef, L, rl, rh)
    assert np.array_equal(_bits(back.cpu().numpy()), _bits(oracle.dwt(want, L, rl, rh, inverse=True)))
    assert np.abs(back.cpu().numpy() - x).max() <= 1e-4 * np.abs(x).max()            # and it is the inverse
    # bf16 input and output
    b = inputs.f32_to_bf16_bits(x)
    xb = torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16)
    coefb, _ = wcc.dwt_fwd(xb, L, dl, dh)
    wantb = oracle.dwt(inputs.bf16_bits_to_f32(b), L, dl, dh)
    assert np.array_equal(_bits(coefb.cpu().numpy()), _bits(wantb))
    backb = wcc.dwt_inv(coefb, L, rl, rh, dtype=torch.bfloat16)
    assert np.array_equal(_bits(backb.float().cpu().numpy()), _bits(oracle.round_bf16(oracle.dwt(wantb, L, rl, rh, inverse=True))))


@pytest.mark.parametrize("name", BANKS)
@pytest.mark.parametrize("cfg", [(2, 12, 20, 32, 64, "f32", 2, 0.25, 8), (1, 40, 24, 32, 32, "bf16", 3, 0.5, 8),
                                 (1, 16, 16, 16, 32, "f32", 2, 0.5, 0)], ids=lambda c: "N%d_%dto%d_%dx%d_%s_L%d_g%s_b%d" % c)
def test_layer_with_other_wavelets(wcc, name, cfg):
    N, Cin, Cout, H, W, dtype, L, gamma, bits = cfg
    bank = wavelets.filter_bank(name)
    w = inputs.custom("wavelet", 43, N, Cin, Cout, H, W, dtype, L, gamma, bits, n_sin=4, fmax=3.0)
    x = torch.from_numpy(w.x.view(np.int16)).cuda().view(torch.bfloat16) if dtype == "bf16" else torch.from_numpy(w.x).cuda()
    y, t = wcc.forward_wavelet(x, torch.from_numpy(w.Wt).cuda(), L, w.k, bits, bank, taps=True)
    assert wcc.last_status() == 0
    want, o = oracle.forward_wavelet(w.x_f32(), w.Wt, L, w.k, bits, *bank, out_bf16=(dtype == "bf16"), taps=True)
    assert np.array_equal(_bits(t["coef"].cpu().numpy()), _bits(o["coef"]))
    assert np.array_equal(t["idx"].cpu().numpy(), o["idx"])
    if bits:
        assert np.array_equal(t["Xq"].cpu().numpy()[:, :Cin], o["Xq"].reshape(-1, Cin))
        assert np.array_equal(t["acc"].cpu().numpy(), o["acc"].reshape(-1, Cout))
        assert np.array_equal(_bits(y.float().cpu().numpy()), _bits(want))
    else:
        assert np.abs(y.float().cpu().numpy() - want).max() <= 2e-2 * np.abs(want).max()

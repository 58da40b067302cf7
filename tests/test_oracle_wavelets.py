"""Pins of the oracle's generic wavelet transform (App. F: WCC with other wavelets) and of the filter banks: Haar taps
reproduce Eq. 3, orthogonal banks are orthonormal (Parseval) and invert exactly, the biorthogonal pair reconstructs
perfectly, Daubechies filters have their vanishing moments, and the layer with Haar taps equals the Haar layer."""
import numpy as np
import pytest

import oracle
from paper_2205_12268_b200 import inputs, wavelets


@pytest.mark.parametrize("name", ["haar", "db2", "db3", "db4", "bior2.2"])
def test_perfect_reconstruction_all_levels(name):
    dl, dh, rl, rh = wavelets.filter_bank(name)
    rng = np.random.default_rng(1)
    x = rng.standard_normal((2, 3, 16, 24))
    for L in (1, 2, 3):
        c = oracle.dwt(x, L, dl.astype(np.float64), dh.astype(np.float64))
        back = oracle.dwt(c, L, rl.astype(np.float64), rh.astype(np.float64), inverse=True)
        assert np.abs(back - x).max() <= 2e-6                       # taps are float32 values
        if name != "bior2.2":                                      # orthogonal: energy is preserved
            assert abs((c * c).sum() - (x * x).sum()) <= 2e-6 * (x * x).sum()


def test_haar_taps_reproduce_eq3():
    dl, dh, _, _ = wavelets.filter_bank("haar")
    rng = np.random.default_rng(2)
    x = rng.standard_normal((1, 2, 8, 16))
    a = oracle.dwt(x, 3, dl.astype(np.float64), dh.astype(np.float64))
    b = oracle.haar_fwd(x, 3)
    assert np.abs(a - b).max() <= 1e-6
    # orientation of the bands: a ramp along the width has its detail in y2 only (one level, interior blocks)
    ramp = np.tile(np.arange(16, dtype=np.float64), (8, 1))[None, None]
    c = oracle.dwt(ramp, 1, dl.astype(np.float64), dh.astype(np.float64))[0, 0]
    assert np.allclose(c[:4, 8:], -1.0, atol=1e-6) and np.allclose(c[4:, :], 0.0, atol=1e-6)


def test_daubechies_filters_from_their_definition():
    r3 = np.sqrt(3.0)
    closed = np.array([1 + r3, 3 + r3, 3 - r3, 1 - r3]) / (4 * np.sqrt(2.0))
    got = wavelets.daubechies(2)
    assert np.allclose(got, closed, atol=1e-12) or np.allclose(got, closed[::-1], atol=1e-12)
    for p in (2, 3, 4, 6):
        lo = wavelets.daubechies(p)
        hi = np.array([(-1) ** t * lo[lo.size - 1 - t] for t in range(lo.size)])
        assert lo.size == 2 * p and abs(lo.sum() - np.sqrt(2.0)) < 1e-10
        for k2 in range(p):                                        # orthonormal to its even shifts
            assert abs((lo[2 * k2:] * lo[:lo.size - 2 * k2]).sum() - (1.0 if k2 == 0 else 0.0)) < 1e-9
        t = np.arange(lo.size, dtype=np.float64)
        for m in range(p):                                         # p vanishing moments of the high-pass filter
            assert abs((hi * t ** m).sum()) < 1e-7 * max(1.0, (np.abs(hi) * t ** m).sum())


def test_smooth_signal_has_small_details_with_more_vanishing_moments():
    """A quadratic along the width is annihilated by db3's high-pass filter (three vanishing moments) away from the
    periodic seam, not by Haar's: the reason the paper tries longer filters."""
    col = np.arange(64, dtype=np.float64)
    x = np.tile(0.01 * col * col, (8, 1))[None, None]
    for name, small in (("haar", False), ("db3", True)):
        dl, dh, _, _ = wavelets.filter_bank(name)
        c = oracle.dwt(x, 1, dl.astype(np.float64), dh.astype(np.float64))[0, 0]
        detail = np.abs(c[:4, 32 + 4:64 - 4]).max()                # y2, interior
        assert (detail < 1e-5) == small


def test_layer_with_haar_taps_is_the_haar_layer():
    w = inputs.custom("wv", 3, 2, 6, 5, 16, 32, "f32", 2, 0.3, 8, n_sin=4, fmax=3.0)
    dl, dh, rl, rh = wavelets.filter_bank("haar")
    y0, t0 = oracle.forward(w.x, w.Wt, 2, w.k, 8, taps=True)
    y1, t1 = oracle.forward_wavelet(w.x, w.Wt, 2, w.k, 8, dl, dh, rl, rh, taps=True)
    assert np.array_equal(t0["idx"], t1["idx"])                    # same selection (norms agree to rounding; no near ties here)
    assert np.abs(t0["Xq"].astype(np.int32) - t1["Xq"].astype(np.int32)).max() <= 1
    assert np.abs(y0 - y1).max() <= 2e-2 * np.abs(y0).max()
    # everything kept, no quantization, any wavelet: the dense 1x1 convolution
    for name in ("db2", "bior2.2"):
        bank = wavelets.filter_bank(name)
        y = oracle.forward_wavelet(w.x, w.Wt, 2, w.P, 0, *bank)
        ref = np.einsum("oc,nchw->nohw", w.Wt.astype(np.float64), w.x.astype(np.float64))
        assert np.abs(y - ref).max() <= 1e-4 * np.abs(ref).max()

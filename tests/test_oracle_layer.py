"""Pins for the oracle's whole layer (Eq. 8-12, Alg. 1): invariants that hold for any correct WCC."""
import numpy as np
import pytest

import oracle
from paper_2205_12268_b200 import inputs


def _dense(Wt, x):
    return np.einsum("oc,nchw->nohw", Wt.astype(np.float64), x.astype(np.float64))


def _maps(seed, N=2, C=5, H=16, W=24):
    return inputs.feature_map(seed, N, C, H, W, n_sin=4, fmax=2.0)


@pytest.mark.parametrize("levels", [1, 2, 3])
def test_keep_everything_equals_dense_conv(levels):
    """T = identity: the layer is the dense 1x1 convolution (the 1x1 conv commutes with H, Eq. 10-12)."""
    x = _maps(1)
    Wt = np.random.default_rng(1).standard_normal((7, 5))
    y = oracle.forward_f64(x, Wt, levels, 16 * 24)
    ref = _dense(Wt, x)
    assert np.abs(y - ref).max() <= 1e-12 * np.abs(ref).max()
    y32 = oracle.forward(x.astype(np.float32), Wt.astype(np.float32), levels, 16 * 24, bits=0)
    ref32 = _dense(Wt.astype(np.float32), x.astype(np.float32))
    assert np.abs(y32 - ref32).max() <= 1e-5 * np.abs(ref32).max()


@pytest.mark.parametrize("k", [1, 37, 192])
def test_fixed_index_set_commutes(k):
    """For the index set I taken from x: WCC(K, x) = H^T T^T T H (K x)  (Eq. 11, same entries extracted)."""
    x = _maps(2)
    Wt = np.random.default_rng(2).standard_normal((3, 5))
    y, t = oracle.forward_f64(x, Wt, 2, k, taps=True)
    Kx = _dense(Wt, x)
    eye = np.eye(3)
    y2 = oracle.forward_f64(Kx, eye, 2, k, idx_in=t["idx"])
    assert np.abs(y - y2).max() <= 1e-12 * np.abs(Kx).max()


def test_dropped_energy_parseval_and_monotone():
    """Identity weights: ||x - WCC_I(x)||^2 is the sum of the norms of the dropped positions (Eq. 8 with an
    orthonormal H), and it cannot grow with k."""
    x = _maps(3, N=2, C=4, H=16, W=16)
    eye = np.eye(4)
    prev = None
    for k in (1, 8, 64, 200, 256):
        y, t = oracle.forward_f64(x, eye, 3, k, taps=True)
        for n in range(2):
            kept = np.zeros(256, bool)
            kept[t["idx"][n]] = True
            err = ((x[n] - y[n]) ** 2).sum()
            drop = t["nrm2"][n][~kept].sum()
            assert abs(err - drop) <= 1e-10 * (x[n] ** 2).sum()
        tot = ((x - y) ** 2).sum()
        assert prev is None or tot <= prev + 1e-12
        prev = tot
    assert prev <= 1e-20 * (x ** 2).sum()          # k = P reproduces x


def test_idempotent_projection():
    x = _maps(4, N=1, C=3, H=16, W=16)
    eye = np.eye(3)
    y, t = oracle.forward_f64(x, eye, 2, 40, taps=True)
    y2, t2 = oracle.forward_f64(y, eye, 2, 40, taps=True)
    assert np.array_equal(t["idx"], t2["idx"])
    assert np.abs(y - y2).max() <= 1e-13 * np.abs(x).max()


def test_selection_is_joint_across_channels():
    """One index list for all channels, ranked by the norm across channels: a channel with a huge
    coefficient at one position forces that position for every channel."""
    x = np.zeros((1, 3, 8, 8))
    x[0, 0] = 1e-3 * np.random.default_rng(5).standard_normal((8, 8))
    x[0, 2, 4:6, 2:4] = np.array([[1, -1], [-1, 1]]) * 50.0       # pure y4 coefficient of block (2, 1)
    y, t = oracle.forward_f64(x, np.eye(3), 1, 1, taps=True)
    assert t["idx"][0].tolist() == [(2 + 4) * 8 + (1 + 4)]          # quadrant layout: y4 at (i+h, j+w)
    assert np.abs(y[0, 2] - x[0, 2]).max() < 1e-12                  # channel 2 kept exactly
    assert np.count_nonzero(y[0, 0]) == 4                           # channel 0 keeps the same single position


def test_quantized_path_taps_are_consistent():
    w = inputs.custom("t", 0, N=2, Cin=6, Cout=5, H=16, W=16, dtype="f32", levels=2, gamma=0.25, bits=8)
    y, t = oracle.forward(w.x, w.Wt, w.levels, w.k, 8, taps=True)
    # indices: the selection of the tapped norms; columns: the tapped coefficients at those indices
    idx, _ = oracle.select_topk(t["nrm2"], w.k)
    assert np.array_equal(idx, t["idx"])
    coef = t["coef"].reshape(2, 6, 256)
    Xc = np.stack([coef[n][:, t["idx"][n]].T for n in range(2)])                 # [N][k][Cin]
    q, s = oracle.quantize(Xc, 8)
    assert np.array_equal(q, t["Xq"]) and s == t["scale_a"][0]                     # one alpha for the whole tensor
    # integer contraction is exact
    acc = np.einsum("oc,nkc->nko", t["Wq"].astype(np.int64), t["Xq"].astype(np.int64))
    assert np.array_equal(acc, t["acc"].astype(np.int64))
    # dequantize, scatter into a zero map, inverse transform
    Y = np.zeros((2, 5, 256), np.float32)
    sc = (t["scale_a"][0] * t["scale_w"]).astype(np.float32)
    for n in range(2):
        Y[n][:, t["idx"][n]] = (t["acc"][n].astype(np.float32) * sc[None, :]).T
    assert np.array_equal(oracle.haar_inv(Y.reshape(2, 5, 16, 16), 2), y)
    # and 8 bits are light: close to the unquantized layer
    yu = oracle.forward(w.x, w.Wt, w.levels, w.k, 0)
    assert np.abs(y - yu).max() < 0.03 * np.abs(yu).max()


def test_fewer_bits_means_larger_error():
    w = inputs.custom("t", 3, N=1, Cin=8, Cout=8, H=16, W=16, dtype="f32", levels=2, gamma=0.5, bits=8)
    yu = oracle.forward(w.x, w.Wt, 2, w.k, 0)
    errs = [np.abs(oracle.forward(w.x, w.Wt, 2, w.k, b) - yu).max() for b in (8, 6, 4)]
    assert errs[0] < errs[1] < errs[2]


def test_bf16_output_rounding():
    w = inputs.custom("t", 4, N=1, Cin=4, Cout=4, H=8, W=8, dtype="bf16", levels=1, gamma=0.5, bits=8)
    y = oracle.forward(w.x_f32(), w.Wt, 1, w.k, 8, out_bf16=False)
    yb = oracle.forward(w.x_f32(), w.Wt, 1, w.k, 8, out_bf16=True)
    assert np.array_equal(yb, oracle.round_bf16(y))
    assert np.all((yb.view(np.uint32) & 0xFFFF) == 0)


def test_layer_rejects_bad_arguments():
    x = np.zeros((1, 2, 8, 8), np.float32)
    Wt = np.zeros((2, 2), np.float32)
    for kw in (dict(levels=1, k=0, bits=8), dict(levels=1, k=65, bits=8), dict(levels=1, k=4, bits=1),
               dict(levels=4, k=4, bits=8)):
        with pytest.raises(ValueError):
            oracle.forward(x, Wt, **kw)

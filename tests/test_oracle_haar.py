"""Pins for the oracle's Haar transform (Eq. 3-6): closed forms, a library convolution with the
printed kernels, an explicit orthonormal matrix, Parseval, exact round trips."""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle


def _read_kernels(golden_dir):
    factor, ker = None, {}
    with open(os.path.join(golden_dir, "eq3_haar_kernels.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = line.split()
            if parts[0] == "factor":
                factor = float(parts[1])
            else:
                ker[parts[0]] = np.array([float(v) for v in parts[1:]], dtype=np.float64).reshape(2, 2)
    w = np.stack([ker["y1"], ker["y2"], ker["y3"], ker["y4"]]) * factor
    return torch.from_numpy(w).reshape(4, 1, 2, 2)


def _one_level(x2d):
    """Quadrants of a 1-level transform of one float64 plane."""
    y = oracle.haar_fwd(x2d[None, None].astype(np.float64), 1)[0, 0]
    h, w = y.shape[0] // 2, y.shape[1] // 2
    return y[:h, :w], y[:h, w:], y[h:, :w], y[h:, w:]


def test_closed_forms_one_level():
    r, c = np.meshgrid(np.arange(8.0), np.arange(8.0), indexing="ij")
    # constant: only the averaging band, doubled
    y1, y2, y3, y4 = _one_level(np.full((8, 8), 3.0))
    assert np.all(y1 == 6.0) and not y2.any() and not y3.any() and not y4.any()
    # ramp along the width: y1 = 4j+1, y2 = -1
    y1, y2, y3, y4 = _one_level(c)
    j = np.arange(4.0)
    assert np.array_equal(y1, np.tile(4 * j + 1, (4, 1)))
    assert np.all(y2 == -1.0) and not y3.any() and not y4.any()
    # ramp along the height: y1 = 4i+1, y3 = -1
    y1, y2, y3, y4 = _one_level(r)
    assert np.array_equal(y1, np.tile((4 * j + 1)[:, None], (1, 4)))
    assert np.all(y3 == -1.0) and not y2.any() and not y4.any()
    # checkerboard: only the diagonal band
    y1, y2, y3, y4 = _one_level((-1.0) ** (r + c))
    assert np.all(y4 == 2.0) and not y1.any() and not y2.any() and not y3.any()


@pytest.mark.parametrize("pos,expect", [((0, 0), (.5, .5, .5, .5)), ((0, 1), (.5, -.5, .5, -.5)),
                                        ((1, 0), (.5, .5, -.5, -.5)), ((1, 1), (.5, -.5, -.5, .5))])
def test_impulses(pos, expect):
    x = np.zeros((8, 8))
    x[pos] = 1.0
    got = tuple(float(q[0, 0]) for q in _one_level(x))
    assert got == expect


def test_constant_multilevel_lowpass():
    for L in (1, 2, 3):
        y = oracle.haar_fwd(np.full((1, 1, 16, 32), 1.25, np.float32), L)[0, 0]
        h, w = 16 >> L, 32 >> L
        assert np.all(y[:h, :w] == 1.25 * 2 ** L)
        y[:h, :w] = 0
        assert not y.any()


@pytest.mark.parametrize("levels", [1, 2, 3])
def test_matches_library_convolution(golden_dir, levels):
    """HWT = stride-2 convolution (cross-correlation, as deep-learning libraries define it) with the
    printed kernels, recursively on y1; iHWT = the transposed convolution."""
    w = _read_kernels(golden_dir)
    rng = np.random.default_rng(1)
    x = rng.standard_normal((2, 3, 16, 24))
    got = oracle.haar_fwd(x, levels)
    ll = torch.from_numpy(x).reshape(6, 1, 16, 24)
    bands = []
    for _ in range(levels):
        y = F.conv2d(ll, w, stride=2)
        bands.append(y[:, 1:4])
        ll = y[:, 0:1]
    # quadrant layout, level by level
    for p in range(6):
        plane = got.reshape(6, 16, 24)[p]
        for l in range(1, levels + 1):
            h, wd = 16 >> l, 24 >> l
            b = bands[l - 1][p].numpy()
            np.testing.assert_allclose(plane[:h, wd:2 * wd], b[0], atol=1e-13)
            np.testing.assert_allclose(plane[h:2 * h, :wd], b[1], atol=1e-13)
            np.testing.assert_allclose(plane[h:2 * h, wd:2 * wd], b[2], atol=1e-13)
        h, wd = 16 >> levels, 24 >> levels
        np.testing.assert_allclose(plane[:h, :wd], ll[p, 0].numpy(), atol=1e-13)
        # concatenated vector of Eq. 6: [y1^L, y2^L, y3^L, y4^L, ..., y2^1, y3^1, y4^1]
        vec = [ll[p, 0].numpy().ravel()]
        for l in range(levels, 0, -1):
            vec += [bands[l - 1][p, i].numpy().ravel() for i in range(3)]
        np.testing.assert_allclose(oracle.concat_order(plane, levels), np.concatenate(vec), atol=1e-13)
    # inverse: transposed convolution, coarsest level first
    rec = ll
    for l in range(levels, 0, -1):
        rec = F.conv_transpose2d(torch.cat([rec, bands[l - 1]], dim=1), w, stride=2)
    np.testing.assert_allclose(oracle.haar_inv(got, levels).reshape(6, 16, 24), rec[:, 0].numpy(), atol=1e-12)


def _level_matrix(H, W, hc, wc):
    """P x P operator of one pyramid level acting on the hc x wc corner (quadrant layout), built from the
    1-D pair [1,1]/sqrt2, [1,-1]/sqrt2 by Kronecker products; identity outside the corner."""
    def a1(n):
        A = np.zeros((n, n))
        s = 1 / np.sqrt(2.0)
        for i in range(n // 2):
            A[i, 2 * i] = s; A[i, 2 * i + 1] = s                    # low  -> first half
            A[n // 2 + i, 2 * i] = s; A[n // 2 + i, 2 * i + 1] = -s   # high -> second half
        return A
    corner = np.kron(a1(hc), a1(wc))          # acts on vec of the corner, row-major
    M = np.eye(H * W)
    ids = (np.arange(hc)[:, None] * W + np.arange(wc)[None, :]).ravel()
    M[np.ix_(ids, ids)] = corner
    return M


@pytest.mark.parametrize("levels", [1, 2, 3])
def test_explicit_orthonormal_matrix(levels):
    H = W = 8
    M = np.eye(H * W)
    for l in range(1, levels + 1):
        M = _level_matrix(H, W, H >> (l - 1), W >> (l - 1)) @ M
    np.testing.assert_allclose(M @ M.T, np.eye(H * W), atol=1e-14)
    rng = np.random.default_rng(2)
    x = rng.standard_normal((1, 1, H, W))
    got = oracle.haar_fwd(x, levels)[0, 0].ravel()
    np.testing.assert_allclose(got, M @ x.ravel(), atol=1e-13)
    np.testing.assert_allclose(oracle.haar_inv(got.reshape(1, 1, H, W), levels).ravel(), M.T @ got, atol=1e-13)


def test_parseval_double():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((2, 5, 32, 64))
    for L in (1, 2, 3, 4):
        y = oracle.haar_fwd(x, L)
        assert abs((y ** 2).sum() / (x ** 2).sum() - 1) < 1e-12
        # per plane too
        np.testing.assert_allclose((y ** 2).sum(axis=(2, 3)), (x ** 2).sum(axis=(2, 3)), rtol=1e-12)


@pytest.mark.parametrize("levels", [1, 2, 3])
def test_dyadic_roundtrip_bit_exact_fp32(levels):
    rng = np.random.default_rng(4)
    x = (rng.integers(-1024, 1025, size=(2, 3, 24, 40)) / 16.0).astype(np.float32)
    y = oracle.haar_fwd(x, levels)
    assert y.dtype == np.float32
    back = oracle.haar_inv(y, levels)
    assert np.array_equal(back.view(np.uint32), x.view(np.uint32))


def test_fp32_tracks_double():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((1, 2, 32, 32))
    y64 = oracle.haar_fwd(x, 3)
    y32 = oracle.haar_fwd(x.astype(np.float32), 3)
    assert np.abs(y32 - y64).max() < 2e-6 * np.abs(y64).max()


def test_bad_shape_rejected():
    with pytest.raises(ValueError):
        oracle.haar_fwd(np.zeros((1, 1, 12, 16), np.float32), 3)    # 12 % 8 != 0

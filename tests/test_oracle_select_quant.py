"""Pins for the oracle's channel norms, joint top-k selection (Alg. 1) and quantizer (Eq. 1-2)."""
import numpy as np
import pytest
import torch

import oracle


# ---------------------------------------------------------------- norms
def test_norms_match_sum_of_squares():
    rng = np.random.default_rng(0)
    c = rng.standard_normal((2, 7, 8, 16))
    np.testing.assert_allclose(oracle.norms(c), (c ** 2).sum(axis=1).reshape(2, -1), rtol=1e-13)
    c32 = c.astype(np.float32)
    np.testing.assert_allclose(oracle.norms(c32), (c32.astype(np.float64) ** 2).sum(axis=1).reshape(2, -1), rtol=2e-6)


def test_norms_exact_on_small_integers():
    rng = np.random.default_rng(1)
    c = rng.integers(-50, 51, size=(1, 9, 4, 4)).astype(np.float32)
    assert np.array_equal(oracle.norms(c), (c.astype(np.int64) ** 2).sum(axis=1).reshape(1, -1).astype(np.float32))


def test_norms_ascending_channel_order_fp32():
    # 4096^2 = 2^24; adding 1 four times in fp32 stays at 2^24 (ties to even) only if the big
    # term comes first; any other order would reach 2^24 + 4.
    c = np.array([4096, 1, 1, 1, 1], np.float32).reshape(1, 5, 1, 1)
    assert oracle.norms(c)[0, 0] == np.float32(16777216.0)
    assert oracle.norms(c[:, ::-1])[0, 0] == np.float32(16777220.0)


def test_norms_fused_multiply_add_fp32():
    # v1^2 = 1 + 2^-11 + 2^-24 is not an fp32 number; a fused step keeps the 2^-24 so that the
    # sum with 2^-24 reaches 1 + 2^-11 + 2^-23, a separate multiply would lose it.
    v0, v1 = np.float32(2.0 ** -12), np.float32(1 + 2.0 ** -12)
    c = np.array([v0, v1], np.float32).reshape(1, 2, 1, 1)
    assert oracle.norms(c)[0, 0] == np.float32(1 + 2.0 ** -11 + 2.0 ** -23)


# ---------------------------------------------------------------- selection
def _brute(nrm, k):
    order = sorted(range(len(nrm)), key=lambda p: (-float(nrm[p]), p))
    return sorted(order[:k]), float(nrm[order[k - 1]])


@pytest.mark.parametrize("seed", range(4))
def test_select_brute_force_random(seed):
    rng = np.random.default_rng(seed)
    P = 16 * 16
    nrm = rng.random((3, P)).astype(np.float32)
    for k in (1, 2, 17, P // 2, P - 1, P):
        idx, tau = oracle.select_topk(nrm, k)
        for n in range(3):
            want, t = _brute(nrm[n], k)
            assert idx[n].tolist() == want
            assert float(tau[n]) == t


def test_select_ties_lowest_index_first():
    # five distinct levels, each repeated many times: every k cuts through a run of equal norms
    rng = np.random.default_rng(7)
    P = 200
    nrm = rng.integers(0, 5, size=(2, P)).astype(np.float32)
    for k in range(1, P + 1, 7):
        idx, tau = oracle.select_topk(nrm, k)
        for n in range(2):
            want, t = _brute(nrm[n], k)
            assert idx[n].tolist() == want and float(tau[n]) == t
    # all equal: the first k positions
    idx, tau = oracle.select_topk(np.ones((1, 64), np.float32), 10)
    assert idx[0].tolist() == list(range(10)) and tau[0] == 1.0
    # duplicated blocks
    blk = rng.random(32).astype(np.float32)
    idx, _ = oracle.select_topk(np.tile(blk, 4)[None], 40)
    assert idx[0].tolist() == _brute(np.tile(blk, 4), 40)[0]


def test_select_output_is_ascending_and_size_k():
    rng = np.random.default_rng(9)
    nrm = rng.random((2, 1000))
    idx, tau = oracle.select_topk(nrm, 123)
    assert idx.shape == (2, 123)
    assert np.all(np.diff(idx, axis=1) > 0)
    for n in range(2):
        kept = np.zeros(1000, bool)
        kept[idx[n]] = True
        assert nrm[n][kept].min() >= nrm[n][~kept].max()
        assert tau[n] == nrm[n][kept].min()


def test_select_rejects_bad_k():
    with pytest.raises(ValueError):
        oracle.select_topk(np.ones((1, 8), np.float32), 0)
    with pytest.raises(ValueError):
        oracle.select_topk(np.ones((1, 8), np.float32), 9)


# ---------------------------------------------------------------- quantizer
def test_quantizer_grid_and_error_bound():
    rng = np.random.default_rng(11)
    x = (rng.standard_normal(5000) * 3).astype(np.float32)
    for bits in (8, 6, 4, 2):
        qmax = 2 ** (bits - 1) - 1
        q, s = oracle.quantize(x, bits)
        assert q.dtype == np.int8 and q.min() >= -qmax and q.max() <= qmax
        assert np.abs(q).max() == qmax                       # the largest magnitude lands on the last level
        assert s == np.float32(np.abs(x).max()) / np.float32(qmax)
        err = np.abs(x.astype(np.float64) - q.astype(np.float64) * float(s))
        assert err.max() <= float(s) / 2 * (1 + 1e-5)


def test_quantizer_round_half_to_even():
    # amax = 127 makes the step exactly 1: half-way inputs must go to the even code
    x = np.array([127, 0.5, 1.5, 2.5, 3.5, -0.5, -1.5, -2.5, 126.5, -126.5, 0.49999997, 0.50000006], np.float32)
    q, s = oracle.quantize(x, 8)
    assert s == 1.0
    assert q.tolist() == [127, 0, 2, 2, 4, 0, -2, -2, 126, -126, 0, 1]


def test_quantizer_is_the_textbook_symmetric_int8():
    rng = np.random.default_rng(12)
    x = (rng.standard_normal(20000) * 2).astype(np.float32)
    q, s = oracle.quantize(x, 8)
    ref = torch.quantize_per_tensor(torch.from_numpy(x), float(s), 0, torch.qint8).int_repr().numpy()
    diff = np.abs(q.astype(np.int32) - ref.astype(np.int32))
    assert diff.max() <= 1 and (diff != 0).mean() < 1e-3     # one multiply vs a division: rare half-way cases only


def test_quantizer_zero_tensor():
    q, s = oracle.quantize(np.zeros(16, np.float32), 8)
    assert not q.any() and s == 0.0


def test_weight_quantizer_per_output_channel():
    rng = np.random.default_rng(13)
    Wt = rng.standard_normal((6, 10)).astype(np.float32) * np.arange(1, 7, dtype=np.float32)[:, None]
    Wq, sw = oracle.quantize_weights(Wt, 8)
    for o in range(6):
        q, s = oracle.quantize(Wt[o], 8)
        assert np.array_equal(Wq[o], q) and sw[o] == s
        assert np.abs(Wq[o]).max() == 127
    assert len(set(sw.tolist())) == 6


def test_round_bf16_matches_library():
    rng = np.random.default_rng(14)
    a = (rng.standard_normal(4096) * 10).astype(np.float32)
    a[:4] = [1.00390625, 1.01171875, -1.00390625, 3.0]       # two exact ties (to even: down, up), sign, exact
    want = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(oracle.round_bf16(a), want)

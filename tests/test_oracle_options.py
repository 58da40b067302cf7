"""Pins of the oracle's layer options: a given clipping parameter (Eq. 2), fewer bits for the weights, the residual
connection (Eq. 13) and the ReLU between chained layers.  Each is checked against something other than the oracle's own
code path: crafted inputs with known codes, a library quantizer, the plain layer's output combined by numpy, and the
invariants that tie the options to the plain layer."""
import numpy as np
import torch

import oracle
from paper_2205_12268_b200 import inputs


def _layer(seed=1, N=2, Cin=6, Cout=5, H=16, W=24, gamma=0.3):
    w = inputs.custom("opt", seed, N, Cin, Cout, H, W, "f32", 2, gamma, 8, n_sin=4, fmax=3.0)
    return w


def test_given_alpha_clips_to_the_ends_of_the_grid():
    # alpha = 2: step 2/127; 3.0 and -7.5 lie beyond +-alpha and must take the extreme codes, 2.0 exactly +127
    x = np.array([0.0, 2.0, -2.0, 3.0, -7.5, 1.0, 2.0 / 127, 1.0 / 127, -3.0 / 127], np.float32)
    q, s = oracle.quantize_alpha(x, 2.0, 8)
    assert s == np.float32(2.0) / np.float32(127.0)
    assert q.tolist() == [0, 127, -127, 127, -127, 64, 1, 0, -2]   # 63.5 -> 64 (even), 0.5 -> 0 (even), -1.5 -> -2 (even)
    q4, s4 = oracle.quantize_alpha(x, 2.0, 4)
    assert s4 == np.float32(2.0) / np.float32(7.0)
    assert q4.tolist() == [0, 7, -7, 7, -7, 4, 0, 0, 0]             # 3.5 -> 4 (even)


def test_given_alpha_against_a_library_quantizer():
    rng = np.random.default_rng(3)
    x = (rng.standard_normal(20000) * 2).astype(np.float32)
    alpha = 3.0                                                     # about 13 % of the values clip
    q, s = oracle.quantize_alpha(x, alpha, 8)
    ref = torch.quantize_per_tensor(torch.from_numpy(x), float(s), 0, torch.qint8).int_repr().numpy().astype(np.int32)
    ref = np.clip(ref, -127, 127)                                   # the library's grid has one more negative code
    diff = np.abs(q.astype(np.int32) - ref)
    assert diff.max() <= 1 and (diff != 0).mean() < 1e-3            # one multiply vs a division: rare half-way cases only
    assert (np.abs(q) == 127).mean() > 0.05


def test_alpha_equal_to_the_largest_kept_magnitude_is_the_plain_layer():
    w = _layer()
    y0, t = oracle.forward(w.x, w.Wt, w.levels, w.k, 8, taps=True)
    amax = np.float32(t["scale_a"][0]) * np.float32(127.0)
    kept = np.stack([t["coef"][n].reshape(w.Cin, -1)[:, t["idx"][n]] for n in range(w.N)])
    amax_direct = np.abs(kept).max()
    y1, t1 = oracle.forward(w.x, w.Wt, w.levels, w.k, 8, taps=True, alpha=float(amax_direct))
    assert np.array_equal(t["Xq"], t1["Xq"]) and np.array_equal(t["acc"], t1["acc"])
    assert np.array_equal(y0.view(np.uint32), y1.view(np.uint32))
    assert abs(float(amax) - float(amax_direct)) <= 1e-6 * float(amax_direct)


def test_smaller_alpha_saturates_and_the_output_follows_the_codes():
    w = _layer(seed=2)
    y0, t0 = oracle.forward(w.x, w.Wt, w.levels, w.k, 8, taps=True)
    amax = float(np.float32(t0["scale_a"][0]) * np.float32(127.0))
    y1, t1 = oracle.forward(w.x, w.Wt, w.levels, w.k, 8, taps=True, alpha=amax / 4)
    assert np.array_equal(t0["idx"], t1["idx"])                     # the selection does not depend on the quantizer
    assert (np.abs(t1["Xq"].astype(np.int32)) == 127).sum() > (np.abs(t0["Xq"].astype(np.int32)) == 127).sum()
    assert t1["scale_a"][0] == np.float32(amax / 4) / np.float32(127.0)
    # accumulators are the integer product of the codes, whatever alpha was
    ref = np.einsum("oc,nkc->nko", t1["Wq"].astype(np.int64), t1["Xq"].astype(np.int64))
    assert np.array_equal(ref, t1["acc"].astype(np.int64))


def test_weight_bits_only_change_the_weight_codes():
    w = _layer(seed=4)
    _, t8 = oracle.forward(w.x, w.Wt, w.levels, w.k, 8, taps=True)
    _, t4 = oracle.forward(w.x, w.Wt, w.levels, w.k, 8, taps=True, wbits=4)
    assert np.array_equal(t8["Xq"], t4["Xq"]) and np.array_equal(t8["idx"], t4["idx"])
    wq4, sw4 = oracle.quantize_weights(w.Wt, 4)
    assert np.array_equal(t4["Wq"], wq4) and np.array_equal(t4["scale_w"], sw4)
    assert np.abs(t4["Wq"].astype(np.int32)).max() == 7             # every row's largest weight sits on +-7
    assert (np.abs(t4["Wq"].astype(np.int32)).max(axis=1) == 7).all()


def test_relu_and_residual_are_applied_after_the_inverse_transform():
    w = _layer(seed=5)
    rng = np.random.default_rng(6)
    res = rng.standard_normal((w.N, w.Cout, w.H, w.W)).astype(np.float32)
    y = oracle.forward(w.x, w.Wt, w.levels, w.k, 8)
    assert np.array_equal(oracle.forward(w.x, w.Wt, w.levels, w.k, 8, relu=True), np.maximum(y, np.float32(0)))
    assert np.array_equal(oracle.forward(w.x, w.Wt, w.levels, w.k, 8, residual=res), y + res)
    both = oracle.forward(w.x, w.Wt, w.levels, w.k, 8, residual=res, relu=True)
    assert np.array_equal(both, np.maximum(y + res, np.float32(0)))     # add first, then the non-linearity
    assert (both == 0).any() and (both > 0).any()
    # rounding to bf16 comes last
    b = oracle.forward(w.x, w.Wt, w.levels, w.k, 8, residual=res, relu=True, out_bf16=True)
    assert np.array_equal(b, oracle.round_bf16(both))


def test_identity_block_with_residual_doubles_the_projection():
    """Identity weights, nothing dropped, no quantization, residual = the input: the layer returns x, so the block
    returns 2x (the skip connection of Eq. 13 adds the block's input)."""
    w = inputs.custom("res", 7, 1, 4, 4, 8, 8, "f32", 3, 1.0, 0, n_sin=3, fmax=2.0)
    eye = np.eye(4, dtype=np.float32)
    y = oracle.forward(w.x, eye, 3, 64, 0, residual=w.x)
    assert np.abs(y - 2 * w.x).max() <= 1e-5 * np.abs(w.x).max()


def test_chain_is_a_loop_of_single_layers():
    rng = np.random.default_rng(8)
    w = inputs.custom("chain", 9, 1, 4, 12, 16, 16, "f32", 2, 0.5, 8, n_sin=3, fmax=2.0)
    Ws = [w.Wt, inputs.weights(21, 4, 12), inputs.weights(22, 12, 4)]
    outs = oracle.chain(w.x, Ws, 2, w.k, 8)
    cur = w.x
    for i, Wt in enumerate(Ws):
        cur = oracle.forward(cur, Wt, 2, w.k, 8)
        if i < 2:
            cur = np.maximum(cur, np.float32(0))
        assert np.array_equal(cur, outs[i])
    assert outs[0].min() >= 0 and outs[2].min() < 0                # ReLU between the layers, none after the last


def test_padded_layer_with_everything_kept_is_the_dense_conv():
    """Zero padding commutes with a pointwise convolution that has no bias: on a 13 x 27 map, everything kept and no
    quantization, the padded layer cropped back equals the dense 1x1 convolution of the original map."""
    rng = np.random.default_rng(11)
    x = rng.standard_normal((2, 5, 13, 27)).astype(np.float32)
    Wt = rng.standard_normal((4, 5)).astype(np.float32)
    y = oracle.forward_padded(x, Wt, 3, 16 * 32, 0)
    ref = np.einsum("oc,nchw->nohw", Wt.astype(np.float64), x.astype(np.float64))
    assert y.shape == ref.shape and np.abs(y - ref).max() <= 1e-5 * np.abs(ref).max()
    # sizes that need no padding: the plain layer
    x2 = rng.standard_normal((1, 3, 16, 8)).astype(np.float32)
    W2 = rng.standard_normal((2, 3)).astype(np.float32)
    assert np.array_equal(oracle.forward_padded(x2, W2, 3, 40, 8), oracle.forward(x2, W2, 3, 40, 8))


def test_bitmap_is_the_index_list_in_another_form():
    idx = np.array([[0, 5, 31, 32, 70], [1, 2, 3, 64, 95]], dtype=np.int32)
    bm = oracle.bitmap_of(idx, 96)
    assert bm.shape == (2, 3)
    assert bm[0].tolist() == [(1 << 0) | (1 << 5) | (1 << 31), 1 << 0, 1 << 6]
    assert bm[1].tolist() == [0b1110, 0, (1 << 0) | (1 << 31)]
    back = [np.flatnonzero(np.unpackbits(bm[n].view(np.uint8), bitorder="little")) for n in range(2)]
    assert all(np.array_equal(back[n], idx[n]) for n in range(2))


def test_depthwise_conv_against_the_library_and_closed_forms():
    import torch.nn.functional as F
    rng = np.random.default_rng(14)
    # small integers: every product and sum is exact, so any summation order gives the same bits
    x = rng.integers(-8, 9, (2, 5, 7, 9)).astype(np.float32)
    w = rng.integers(-4, 5, (5, 3, 3)).astype(np.float32)
    ref = F.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double()[:, None], padding=1, groups=5).numpy()
    assert np.array_equal(oracle.dwconv3x3(x, w).astype(np.float64), ref)
    # real values: within rounding of the double result
    x = rng.standard_normal((1, 3, 16, 12)).astype(np.float32)
    w = rng.standard_normal((3, 3, 3)).astype(np.float32)
    ref = F.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double()[:, None], padding=1, groups=3).numpy()
    assert np.abs(oracle.dwconv3x3(x, w) - ref).max() <= 1e-5 * np.abs(ref).max()
    # a kernel with a single 1 at tap (i, j) shifts the map by (1 - i, 1 - j) with zeros moving in: orientation of the taps
    x = np.arange(20, dtype=np.float32).reshape(1, 1, 4, 5)
    w = np.zeros((1, 3, 3), np.float32); w[0, 0, 2] = 1        # out[r][c] = x[r-1][c+1]
    y = oracle.dwconv3x3(x, w)[0, 0]
    assert y[0].tolist() == [0] * 5 and y[1].tolist() == [1, 2, 3, 4, 0] and y[3].tolist() == [11, 12, 13, 14, 0]
    w = np.zeros((1, 3, 3), np.float32); w[0, 1, 1] = 1        # identity
    assert np.array_equal(oracle.dwconv3x3(x, w), x)


def test_block_with_identity_parts_returns_twice_the_input():
    """Identity pointwise weights, identity depthwise kernel, everything kept, no quantization: every part is the
    identity, so the block returns x + x (the skip connection of Eq. 13)."""
    w = inputs.custom("blk", 15, 1, 4, 4, 8, 16, "f32", 3, 1.0, 0, n_sin=3, fmax=2.0)
    eye = np.eye(4, dtype=np.float32)
    dw = np.zeros((4, 3, 3), np.float32); dw[:, 1, 1] = 1
    y = oracle.block(w.x, eye, dw, eye, 3, 128, 0)
    assert np.abs(y - 2 * w.x).max() <= 1e-5 * np.abs(w.x).max()
    # and with real parts it is the composition of its three steps plus the input
    rng = np.random.default_rng(16)
    W1, W3 = inputs.weights(1, 12, 4), inputs.weights(2, 4, 12)
    dw = rng.standard_normal((12, 3, 3)).astype(np.float32)
    y, t = oracle.block(w.x, W1, dw, W3, 3, 40, 8, taps=True)
    assert np.array_equal(t["u"], oracle.forward(w.x, W1, 3, 40, 8))
    assert np.array_equal(t["v"], oracle.dwconv3x3(t["u"], dw))
    assert np.array_equal(y, oracle.forward(t["v"], W3, 3, 40, 8) + w.x)

"""GPU parity of the layer options (wcc_forward_ex) and of the chain entry point (wcc_chain_forward) against the
CPU oracle: a given clipping parameter that saturates (codes, accumulators and output bit for bit), 4-bit weights,
residual add and ReLU on the way out, weights quantized ahead of the call, and the six-layer chain workload."""
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


def _x_dev(w):
    if w.dtype == "bf16":
        return torch.from_numpy(w.x.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(w.x).cuda()


def _res(w, seed):
    r = np.random.default_rng(seed).standard_normal((w.N, w.Cout, w.H, w.W)).astype(np.float32)
    if w.dtype == "bf16":
        b = inputs.f32_to_bf16_bits(r)
        return torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16), inputs.bf16_bits_to_f32(b)
    return torch.from_numpy(r).cuda(), r


def _bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


CASES = [  # N, Cin, Cout, H, W, dtype, levels, gamma
    (2, 12, 20, 32, 64, "f32", 2, 0.25),
    (2, 40, 24, 16, 64, "bf16", 3, 0.5),
    (1, 24, 144, 32, 64, "bf16", 3, 0.25),       # several chunks of output channels
    (1, 6, 4, 4, 6, "f32", 1, 0.5),              # rows the TMA path cannot take: the one-tile kernel
    (3, 70, 20, 16, 64, "f32", 1, 0.4),
]


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: "N%d_%dto%d_%dx%d_%s_L%d_g%s" % c)
def test_given_alpha_saturates_like_the_oracle(wcc, cfg):
    N, Cin, Cout, H, W, dtype, L, gamma = cfg
    w = inputs.custom("alpha", 21, N, Cin, Cout, H, W, dtype, L, gamma, 8, n_sin=4, fmax=3.0)
    x, Wt = _x_dev(w), torch.from_numpy(w.Wt).cuda()
    _, t0 = oracle.forward(w.x_f32(), w.Wt, L, w.k, 8, out_bf16=(dtype == "bf16"), taps=True)
    amax = float(np.float32(t0["scale_a"][0]) * np.float32(127.0))
    for alpha in (amax / 3, amax * 1.7):              # one that clips many kept coefficients, one that clips none
        want, o = oracle.forward(w.x_f32(), w.Wt, L, w.k, 8, out_bf16=(dtype == "bf16"), taps=True, alpha=alpha)
        y, t = wcc.forward(x, Wt, L, w.k, 8, taps=True, alpha=alpha)
        assert wcc.last_status() == 0
        M = w.N * w.k
        assert np.array_equal(t["idx"].cpu().numpy(), o["idx"])
        assert np.array_equal(t["Xq"].cpu().numpy()[:, :Cin], o["Xq"].reshape(M, Cin))
        assert np.array_equal(t["acc"].cpu().numpy(), o["acc"].reshape(M, Cout))
        assert t["scale_a"].cpu().numpy().view(np.uint32)[0] == o["scale_a"].view(np.uint32)[0]
        assert np.array_equal(_bits(y.float().cpu().numpy()), _bits(want))
    assert (np.abs(oracle.forward(w.x_f32(), w.Wt, L, w.k, 8, taps=True, alpha=amax / 3)[1]["Xq"].astype(np.int32)) == 127).sum() > 10


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: "N%d_%dto%d_%dx%d_%s_L%d_g%s" % c)
def test_residual_relu_and_four_bit_weights(wcc, cfg):
    N, Cin, Cout, H, W, dtype, L, gamma = cfg
    w = inputs.custom("opts", 22, N, Cin, Cout, H, W, dtype, L, gamma, 8, n_sin=4, fmax=3.0)
    x, Wt = _x_dev(w), torch.from_numpy(w.Wt).cuda()
    res_d, res_h = _res(w, 5)
    bf = dtype == "bf16"
    for kw in (dict(relu=True), dict(residual=True), dict(residual=True, relu=True), dict(wbits=4),
               dict(wbits=4, residual=True, relu=True, alpha=0.9)):
        okw = dict(kw)
        gkw = dict(kw)
        if kw.get("residual"):
            okw["residual"], gkw["residual"] = res_h, res_d
        want, o = oracle.forward(w.x_f32(), w.Wt, L, w.k, 8, out_bf16=bf, taps=True, **okw)
        y, t = wcc.forward(x, Wt, L, w.k, 8, taps=True, **gkw)
        assert wcc.last_status() == 0
        assert np.array_equal(t["Wq"].cpu().numpy()[:, :Cin], o["Wq"])
        assert np.array_equal(t["scale_w"].cpu().numpy().view(np.uint32), o["scale_w"].view(np.uint32))
        assert np.array_equal(t["acc"].cpu().numpy(), o["acc"].reshape(-1, Cout))
        assert np.array_equal(_bits(y.float().cpu().numpy()), _bits(want)), kw
        y2 = wcc.forward(x, Wt, L, w.k, 8, **gkw)                      # without taps: same bytes
        assert torch.equal(y, y2)


def test_residual_may_be_the_output_buffer(wcc):
    w = inputs.custom("inplace", 23, 2, 16, 16, 32, 64, "f32", 3, 0.3, 8, n_sin=4, fmax=3.0)
    x, Wt = _x_dev(w), torch.from_numpy(w.Wt).cuda()
    want = oracle.forward(w.x, w.Wt, 3, w.k, 8, residual=w.x)          # y = x + WCC(x): the skip connection of Eq. 13
    y = x.clone()
    wcc.forward(x, Wt, 3, w.k, 8, y=y, residual=y)
    assert wcc.last_status() == 0
    assert np.array_equal(_bits(y.cpu().numpy()), _bits(want))


def test_weights_quantized_ahead_of_the_call(wcc):
    w = inputs.custom("preq", 24, 2, 40, 24, 16, 64, "bf16", 3, 0.5, 8, n_sin=4, fmax=3.0)
    x, Wt = _x_dev(w), torch.from_numpy(w.Wt).cuda()
    y0, t = wcc.forward(x, Wt, 3, w.k, 8, taps=True)
    y1 = wcc.forward(x, None, 3, w.k, 8, Wq=t["Wq"].clone(), scale_w=t["scale_w"].clone())
    assert wcc.last_status() == 0
    assert torch.equal(y0, y1)
    # codes built on the host from the oracle's quantizer work just as well
    kp = wcc.kpad(w.Cin, 8)
    q, s = oracle.quantize_weights(w.Wt, 8)
    qp = np.zeros((w.Cout, kp), np.int8)
    qp[:, :w.Cin] = q
    y2 = wcc.forward(x, None, 3, w.k, 8, Wq=torch.from_numpy(qp).cuda(), scale_w=torch.from_numpy(s).cuda())
    assert torch.equal(y0, y2)


def test_option_errors_come_back_before_any_launch(wcc):
    x = torch.zeros((1, 8, 16, 16), device="cuda")
    Wt = torch.zeros((8, 8), device="cuda")
    for kw, code in ((dict(wbits=9), 4), (dict(wbits=4, bits=0), 4), (dict(alpha=float("inf")), 2)):
        bits = kw.pop("bits", 8)
        with pytest.raises(wcc.WccError) as e:
            wcc.forward(x, Wt, 2, 64, bits, **kw)
        assert e.value.code == code
    with pytest.raises(wcc.WccError) as e:
        wcc.forward(x, None, 2, 64, 8, Wq=torch.zeros((8, 32), dtype=torch.int8, device="cuda"), scale_w=None, relu=True)
    assert e.value.code == 1


def _chain_case(wcc, N, H, W, L, gamma, dtype, alphas=None, relu_last=False):
    first = inputs.custom("chain", 0, N, 32, 192, H, W, dtype, L, gamma, 8, n_sin=16, fmax=8.0)
    chans = [32, 192, 32, 192, 32, 192, 32]
    Ws = [inputs.weights(100 + i, chans[i + 1], chans[i]) for i in range(6)]
    x = _x_dev(first)
    ch = wcc.Chain(x, [torch.from_numpy(a).cuda() for a in Ws], L, first.k, 8, relu_last=relu_last, alphas=alphas)
    y = ch(x)
    assert wcc.last_status() == 0
    outs = oracle.chain(first.x_f32(), Ws, L, first.k, 8, out_bf16=(dtype == "bf16"), relu_last=relu_last, alphas=alphas)
    assert np.array_equal(_bits(y.float().cpu().numpy()), _bits(outs[-1]))
    y2 = ch(x)                                                        # the workspace is reusable as it is
    assert torch.equal(y, y2)
    return outs


def test_chain_small(wcc):
    _chain_case(wcc, 2, 64, 128, 3, 0.25, "bf16")
    _chain_case(wcc, 1, 32, 64, 2, 0.5, "f32", relu_last=True)
    _chain_case(wcc, 2, 32, 64, 3, 0.25, "bf16", alphas=[2.0, 3.0, 2.5, 3.0, 2.5, 3.0])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("L", [1, 2, 3])
def test_chain_with_odd_channel_counts(wcc, dtype, L):
    """Channel counts that are no multiples of eight, a single group of output channels, several chunks of 32, ragged
    tile groups: every layer's second pass also produces the next layer's norms, and the end result must still equal
    the oracle's loop of single layers (which it can only do if every intermediate norm, threshold and scale did)."""
    chans = [12, 20, 7, 40, 100, 9, 33]
    N, H, W = 3, 24, 72
    w0 = inputs.custom("oddchain", 60 + L, N, chans[0], chans[1], H, W, dtype, L, 0.3, 8, n_sin=4, fmax=3.0)
    Ws = [inputs.weights(200 + i, chans[i + 1], chans[i]) for i in range(len(chans) - 1)]
    x = _x_dev(w0)
    for alphas in (None, [1.5, 0.0, 2.0, 0.0, 1.0, 0.0]):
        ch = wcc.Chain(x, [torch.from_numpy(a).cuda() for a in Ws], L, w0.k, 8, alphas=alphas)
        y = ch(x)
        assert wcc.last_status() == 0
        outs = oracle.chain(w0.x_f32(), Ws, L, w0.k, 8, out_bf16=(dtype == "bf16"), alphas=alphas)
        assert np.array_equal(_bits(y.float().cpu().numpy()), _bits(outs[-1]))
        assert torch.equal(y, ch(x))


def test_chain_full_size(wcc):
    """The six-layer chain workload as the benchmark runs it: 2 x 256 x 512 bf16, three levels, a quarter kept."""
    outs = _chain_case(wcc, 2, 256, 512, 3, 0.25, "bf16")
    assert all(o.min() >= 0 for o in outs[:-1]) and outs[-1].min() < 0

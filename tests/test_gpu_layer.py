"""GPU parity of the whole layer (wcc_forward / wcc_forward_debug) against the CPU oracle on the same seeded
inputs.  Kept indices, int8 codes and int32 accumulators must be identical; the floating-point output must be
within 1e-4 (fp32 activations) or 2e-2 (bf16 activations, and the unquantized bf16 contraction) of the
output's largest magnitude."""
import numpy as np
import pytest
import torch

import oracle
from paper_2205_12268_b200 import inputs

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 2e-2}


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


def _run_and_compare(wcc, w, staged=False):
    x = _x_dev(w)
    Wt = torch.from_numpy(w.Wt).cuda()
    ws = wcc.Workspace.for_problem(x, w.Cout, w.levels, w.k, w.bits, staged=staged)
    ws.buf.fill_(0xFF)                                        # poison: nothing may depend on old contents
    y, t = wcc.forward(x, Wt, w.levels, w.k, w.bits, ws=ws, taps=True, staged=staged)
    assert wcc.last_status() == 0
    want, o = oracle.forward(w.x_f32(), w.Wt, w.levels, w.k, w.bits, out_bf16=(w.dtype == "bf16"), taps=True)

    P, M = w.P, w.N * w.k
    assert np.array_equal(t["coef"].cpu().numpy().view(np.uint32), o["coef"].reshape(w.N, w.Cin, P).view(np.uint32))
    assert np.array_equal(t["nrm2"].cpu().numpy().view(np.uint32), o["nrm2"].view(np.uint32))
    assert np.array_equal(t["idx"].cpu().numpy(), o["idx"])
    if w.bits >= 2:
        kp = wcc.kpad(w.Cin, w.bits)
        Xq = t["Xq"].cpu().numpy()
        assert np.array_equal(Xq[:, :w.Cin], o["Xq"].reshape(M, w.Cin))
        assert not Xq[:, w.Cin:].any() and Xq.shape[1] == kp
        Wq = t["Wq"].cpu().numpy()
        assert np.array_equal(Wq[:, :w.Cin], o["Wq"]) and not Wq[:, w.Cin:].any()
        assert np.array_equal(t["scale_w"].cpu().numpy().view(np.uint32), o["scale_w"].view(np.uint32))
        assert t["scale_a"].cpu().numpy().view(np.uint32)[0] == o["scale_a"].view(np.uint32)[0]
        assert np.array_equal(t["acc"].cpu().numpy(), o["acc"].reshape(M, w.Cout))
    else:
        cols = np.stack([o["coef"].reshape(w.N, w.Cin, P)[n][:, o["idx"][n]].T for n in range(w.N)]).reshape(M, w.Cin)
        Xb = t["Xb"].float().cpu().numpy()
        assert np.array_equal(Xb[:, :w.Cin], oracle.round_bf16(cols)) and not Xb[:, w.Cin:].any()
        prod = t["acc"].view(torch.float32).cpu().numpy().astype(np.float64)
        ref = cols.astype(np.float64) @ w.Wt.astype(np.float64).T
        assert np.abs(prod - ref).max() <= 2e-2 * np.abs(ref).max()

    got = y.float().cpu().numpy()
    scale = np.abs(want).max()
    tol = 2e-2 if w.bits == 0 else TOL[w.dtype]
    err = np.abs(got - want).max()
    assert err <= tol * scale, (err, scale)
    if w.bits >= 2:
        # same integers and the same fp32 operation order: identical up to the final rounding to the output type
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # plain wcc_forward gives the same bytes as the debug entry point, and does so again (determinism)
    y2 = wcc.forward(x, Wt, w.levels, w.k, w.bits, ws=ws, staged=staged)
    y3 = wcc.forward(x, Wt, w.levels, w.k, w.bits, staged=staged)
    assert torch.equal(y, y2) and torch.equal(y, y3)
    assert wcc.last_status() == 0
    return got, want


SMALL = [  # N, Cin, Cout, H, W, dtype, levels, gamma, bits
    (1, 3, 5, 8, 8, "f32", 3, 0.5, 8),
    (2, 6, 4, 16, 24, "f32", 1, 0.3, 8),
    (2, 6, 4, 16, 24, "bf16", 2, 0.3, 8),
    (1, 2, 2, 4, 6, "f32", 1, 0.5, 8),            # W % 4 == 2
    (3, 33, 17, 32, 72, "bf16", 3, 0.2, 8),       # ragged tile, odd channel counts
    (2, 130, 24, 16, 64, "f32", 2, 0.5, 8),       # two K atoms
    (1, 24, 144, 64, 64, "bf16", 3, 0.25, 8),
    (1, 256, 256, 16, 32, "f32", 3, 0.6, 8),      # largest channel counts
    (2, 16, 40, 40, 200, "f32", 3, 1.0, 8),       # keep everything
    (2, 16, 8, 40, 200, "bf16", 3, 0.001, 8),     # keep almost nothing (k = 8 < one row tile)
    (1, 20, 36, 32, 32, "f32", 2, 0.25, 0),       # unquantized bf16 contraction
    (2, 144, 24, 32, 64, "bf16", 3, 0.5, 0),
    (1, 8, 8, 32, 32, "f32", 2, 0.25, 4),         # fewer bits on the same int8 path
    (1, 8, 8, 32, 32, "f32", 2, 0.25, 2),
    (1, 40, 24, 8, 96, "bf16", 3, 0.5, 8),        # three tiles: the last group of four is ragged
    (3, 12, 80, 16, 160, "f32", 2, 0.3, 8),       # output channels in chunks of 32, 32 and 16; 15 tiles
    (2, 70, 20, 16, 64, "bf16", 3, 0.4, 8),       # three K steps streamed through two operand buffers
    (1, 20, 100, 24, 64, "bf16", 3, 0.3, 0),      # unquantized, several chunks of output channels, two K steps
]


@pytest.mark.parametrize("staged", [False, True], ids=["fused", "staged"])
@pytest.mark.parametrize("cfg", SMALL, ids=lambda c: "N%d_%dto%d_%dx%d_%s_L%d_g%s_b%d" % c)
def test_layer_small(wcc, cfg, staged):
    N, Cin, Cout, H, W, dtype, L, gamma, bits = cfg
    w = inputs.custom("small", 3, N, Cin, Cout, H, W, dtype, L, gamma, bits, n_sin=4, fmax=3.0)
    _run_and_compare(wcc, w, staged=staged)


@pytest.mark.parametrize("staged", [False, True], ids=["fused", "staged"])
def test_layer_image_larger_than_one_cluster(wcc, staged):
    """More positions per image (512 x 512) than the cluster select holds in registers: the cooperative select runs and
    the fused second pass takes its keep / drop decisions from the rank map."""
    w = inputs.custom("large", 9, 1, 4, 6, 512, 512, "f32", 3, 0.1, 8, n_sin=6, fmax=6.0)
    _run_and_compare(wcc, w, staged=staged)


def test_layer_partial_ties_at_the_threshold(wcc):
    """Many positions share the k-th norm exactly and only some of them are kept (lowest positions first): the select
    must fall back to the ordered compaction and the second pass to the rank map."""
    w = inputs.custom("ties", 2, 2, 3, 5, 32, 64, "f32", 2, 0.5, 8, n_sin=3, fmax=2.0)
    blk = w.x[:, :, :4, :4].copy()                           # one 4x4 block (a whole level-2 unit) tiled over the map
    w.x[:] = np.tile(blk, (1, 1, 8, 16))
    for k in (1, 100, 777, 1024, 2047):
        w.k = k
        _run_and_compare(wcc, w)


@pytest.mark.parametrize("distinct", [False, True], ids=["equal", "distinct"])
def test_layer_threshold_bin_holds_more_keys_than_can_be_ranked(wcc, distinct):
    """Thousands of norms fall into the histogram bin of the threshold (a 2x2 block tiled over a 128x128 map gives four
    norm values, 4096 positions each; with `distinct` every position also gets a tiny relative perturbation, so the keys
    of a bin differ in their low bits): the select cannot rank that many candidates directly and has to run its digit
    rounds on top of the first pass's histogram.  k cuts through such a bin, through a run of equal keys, and lands on
    its ends."""
    w = inputs.custom("crowd", 4, 2, 3, 5, 128, 128, "f32", 1, 0.5, 8, n_sin=3, fmax=2.0)
    blk = w.x[:, :, :2, :2].copy()
    w.x[:] = np.tile(blk, (1, 1, 64, 64))
    if distinct:
        rng = np.random.default_rng(11)
        w.x *= (1.0 + 1e-4 * rng.standard_normal(w.x.shape)).astype(np.float32)
    for k in (1, 3000, 4096, 4097, 9000, 16383):
        w.k = k
        _run_and_compare(wcc, w)


def test_layer_k_equals_one_and_all(wcc):
    for k in (1, 16 * 16):
        w = inputs.custom("edge", 5, 2, 5, 7, 16, 16, "f32", 2, 0.5, 8, k=k)
        _run_and_compare(wcc, w)


def test_layer_zero_input(wcc):
    w = inputs.custom("zero", 0, 1, 4, 4, 8, 8, "f32", 1, 0.5, 8)
    w.x[:] = 0
    got, want = _run_and_compare(wcc, w)
    assert not got.any()


def test_keep_everything_unquantized_is_the_dense_conv(wcc):
    w = inputs.custom("dense", 7, 2, 16, 24, 32, 32, "f32", 3, 1.0, 0)
    y = wcc.forward(torch.from_numpy(w.x).cuda(), torch.from_numpy(w.Wt).cuda(), 3, w.k, 0).cpu().numpy()
    ref = np.einsum("oc,nchw->nohw", w.Wt.astype(np.float64), w.x.astype(np.float64))
    assert np.abs(y - ref).max() <= 2e-2 * np.abs(ref).max()


@pytest.mark.parametrize("staged", [False, True], ids=["fused", "staged"])
@pytest.mark.parametrize("name", ["C1", "C2", "C3", "C3u", "C4", "C4b", "C5a", "C5b"])
def test_layer_named_workloads_full_size(wcc, name, staged):
    """The five benchmark workloads at full size, in the launch configuration the bench times."""
    _run_and_compare(wcc, inputs.make(name), staged=staged)


@pytest.mark.parametrize("name,batch", [("C4", 24), ("C2", 16)], ids=["C4x24", "C2x16"])
def test_layer_profiled_batches_full_size(wcc, name, batch):
    """The batches the DRAM counters are taken on (the named workload with more images, so that x exceeds the L2):
    several waves of every kernel, the first pass walking more than one tile per CTA."""
    _run_and_compare(wcc, inputs.make(name, N=batch))


def _random_shapes(count, seed):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(count):
        L = int(rng.integers(1, 4))
        unit = 1 << L
        H = unit * int(rng.integers(1, 6))
        W = unit * int(rng.integers(1, 24))
        if L == 1 and rng.random() < 0.7:
            W = 4 * max(1, W // 4)                                    # mostly the vectorized paths
        cfg = (int(rng.integers(1, 4)), int(rng.integers(1, 80)), int(rng.integers(1, 100)), H, W,
               "bf16" if rng.random() < 0.5 else "f32", L, float(rng.choice([0.05, 0.125, 0.25, 0.5, 0.9])),
               int(rng.choice([8, 8, 8, 0, 5])))
        out.append(cfg)
    return out


@pytest.mark.parametrize("cfg", _random_shapes(24, 2205), ids=lambda c: "N%d_%dto%d_%dx%d_%s_L%d_g%s_b%d" % c)
def test_layer_random_shapes(wcc, cfg):
    """Seeded random small shapes (channel counts, tile counts, levels, types, keep ratios, bit widths drawn at random):
    every intermediate and the output against the oracle, as for the hand-picked shapes above."""
    N, Cin, Cout, H, W, dtype, L, gamma, bits = cfg
    w = inputs.custom("fuzz", 11, N, Cin, Cout, H, W, dtype, L, gamma, bits, n_sin=4, fmax=3.0)
    _run_and_compare(wcc, w)


def test_bench_workload_as_cuda_graph_replay(wcc):
    """The launch configuration the benchmark times: wcc_forward of workload C2 captured once in a CUDA graph and
    replayed (with the L2 cache overwritten in between); every replay must give the oracle's output bit for bit."""
    w = inputs.make("C2")
    x = _x_dev(w)
    Wt = torch.from_numpy(w.Wt).cuda()
    y = torch.empty((w.N, w.Cout, w.H, w.W), dtype=x.dtype, device="cuda")
    ws = wcc.Workspace.for_problem(x, w.Cout, w.levels, w.k, w.bits)
    wcc.forward(x, Wt, w.levels, w.k, w.bits, y=y, ws=ws)          # sets kernel attributes outside the capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        wcc.forward(x, Wt, w.levels, w.k, w.bits, y=y, ws=ws)
    torch.cuda.current_stream().wait_stream(side)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        wcc.forward(x, Wt, w.levels, w.k, w.bits, y=y, ws=ws)
    want = oracle.forward(w.x_f32(), w.Wt, w.levels, w.k, w.bits, out_bf16=True)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for rep in range(3):
        y.fill_(float("nan"))
        ws.buf.fill_(0xFF)                                          # nothing may depend on what the last replay left
        flush.fill_(rep)
        g.replay()
        torch.cuda.synchronize()
        assert np.array_equal(y.float().cpu().numpy().view(np.uint32), want.view(np.uint32))
    assert wcc.last_status() == 0


def _chain(wcc, N, H, W, L, gamma):
    first = inputs.custom("chain", 0, N, 32, 192, H, W, "bf16", L, gamma, 8, n_sin=16, fmax=8.0)
    x = _x_dev(first)
    chans = [32, 192, 32, 192, 32, 192, 32]
    for i in range(6):
        Wt_np = inputs.weights(100 + i, chans[i + 1], chans[i])
        y = wcc.forward(x, torch.from_numpy(Wt_np).cuda(), L, first.k, 8)
        want = oracle.forward(x.float().cpu().numpy(), Wt_np, L, first.k, 8, out_bf16=True)
        assert np.array_equal(y.float().cpu().numpy().view(np.uint32), want.view(np.uint32)), i
        x = torch.relu(y)
    assert wcc.last_status() == 0


def test_chain_of_layers_with_relu(wcc):
    """Six pointwise WCC layers 32 -> 192 -> 32 ... with ReLU in between (reduced spatial size); each layer
    is checked against the oracle fed with the GPU's own input to that layer."""
    _chain(wcc, 2, 64, 128, 3, 0.25)


def test_chain_of_layers_with_relu_full_size(wcc):
    """The same chain at the benchmark's size (2 x 256 x 512)."""
    _chain(wcc, 2, 256, 512, 3, 0.25)


_C5_CACHE = {}


def _c5_workload(cin, cout):
    """The two layer shapes of the six-layer chain workload at full size (inputs generated once per shape)."""
    if (cin, cout) not in _C5_CACHE:
        _C5_CACHE[(cin, cout)] = inputs.custom("C5", 0, 2, cin, cout, 256, 512, "bf16", 3, 0.25, 8, n_sin=16, fmax=8.0)
    return _C5_CACHE[(cin, cout)]


@pytest.mark.parametrize("gamma", [0.5, 0.25, 0.125, 0.0625], ids=lambda g: "g%s" % g)
@pytest.mark.parametrize("L", [1, 2, 3], ids=lambda l: "L%d" % l)
@pytest.mark.parametrize("shape", [(32, 192), (192, 32)], ids=lambda c: "%dto%d" % c)
def test_layer_config5_sweep_full_size(wcc, shape, L, gamma):
    """Every (levels, keep ratio) point of the chain workload's sweep, both layer shapes, 2 x 256 x 512 bf16: output
    bit for bit against the oracle; at the 1/16 points also every intermediate (many accumulator chunks per tile group
    at one and two levels, where a tile is a thin strip of the image)."""
    import copy
    w = copy.copy(_c5_workload(*shape))
    w.levels = L
    w.k = inputs.keep_count(gamma, w.P)
    if gamma == 0.0625:
        _run_and_compare(wcc, w)
        return
    x = _x_dev(w)
    y = wcc.forward(x, torch.from_numpy(w.Wt).cuda(), L, w.k, 8)
    assert wcc.last_status() == 0
    want = oracle.forward(w.x_f32(), w.Wt, L, w.k, 8, out_bf16=True)
    assert np.array_equal(y.float().cpu().numpy().view(np.uint32), want.view(np.uint32))


def test_workspace_too_small_is_rejected(wcc):
    x = torch.zeros((1, 4, 8, 8), device="cuda")
    Wt = torch.zeros((4, 4), device="cuda")
    ws = wcc.Workspace(512, x.device)
    with pytest.raises(wcc.WccError) as e:
        wcc.forward(x, Wt, 1, 8, 8, ws=ws)
    assert e.value.code == 7

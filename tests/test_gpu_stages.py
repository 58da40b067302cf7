"""GPU parity of the single stages (wcc_haar_fwd, wcc_haar_inv, wcc_select_topk) against the CPU oracle,
through the C ABI.  Integer and index results must be identical; the fp32 transforms follow the same
operation order as the oracle and must be bit-identical too."""
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


def _bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def _to_dev(x, dtype):
    if dtype == "bf16":
        b = inputs.f32_to_bf16_bits(x)
        return torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16), inputs.bf16_bits_to_f32(b)
    return torch.from_numpy(x).cuda(), x


SHAPES = [  # N, C, H, W, levels
    (1, 3, 8, 8, 3), (1, 1, 2, 2, 1), (1, 2, 4, 6, 1), (2, 5, 16, 24, 1), (2, 5, 16, 24, 2), (2, 5, 16, 24, 3),
    (2, 3, 32, 72, 3), (1, 4, 64, 320, 2), (1, 7, 6, 130, 1), (3, 9, 40, 200, 3), (1, 33, 128, 256, 3), (2, 17, 96, 320, 2),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", SHAPES)
def test_haar_fwd_and_norms_bit_exact(wcc, shape, dtype):
    N, Cc, H, W, L = shape
    x = inputs.feature_map(11, N, Cc, H, W, 4, 3.0).astype(np.float32)
    xd, xh = _to_dev(x, dtype)
    coef, nrm2 = wcc.haar_fwd(xd, L)
    assert wcc.last_status() == 0
    want = oracle.haar_fwd(xh, L)
    assert np.array_equal(_bits(coef.cpu().numpy()), _bits(want))
    assert np.array_equal(_bits(nrm2.cpu().numpy()), _bits(oracle.norms(want)))
    coef2, none = wcc.haar_fwd(xd, L, want_norms=False)
    assert none is None and torch.equal(coef, coef2)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", SHAPES)
def test_haar_inv_bit_exact(wcc, shape, dtype):
    N, Cc, H, W, L = shape
    rng = np.random.default_rng(5)
    coef = rng.standard_normal((N, Cc, H, W)).astype(np.float32)
    out = wcc.haar_inv(torch.from_numpy(coef).cuda(), L, torch.bfloat16 if dtype == "bf16" else torch.float32)
    want = oracle.haar_inv(coef, L)
    if dtype == "bf16":
        want = oracle.round_bf16(want)
    assert np.array_equal(_bits(out.float().cpu().numpy()), _bits(want))


def test_haar_roundtrip_dyadic_exact(wcc):
    rng = np.random.default_rng(6)
    x = (rng.integers(-1024, 1025, size=(2, 3, 64, 96)) / 16.0).astype(np.float32)
    xd = torch.from_numpy(x).cuda()
    for L in (1, 2, 3):
        coef, _ = wcc.haar_fwd(xd, L)
        assert torch.equal(wcc.haar_inv(coef, L), xd)


def _check_select(wcc, nrm, k):
    idx, tau = wcc.select_topk(torch.from_numpy(nrm).cuda(), k)
    assert wcc.last_status() == 0
    widx, wtau = oracle.select_topk(nrm, k)
    assert np.array_equal(idx.cpu().numpy(), widx)
    assert np.array_equal(tau.cpu().numpy(), wtau)          # by value: -0 and +0 rank equal


@pytest.mark.parametrize("P", [64, 100, 2048, 2049, 5000, 32768, 131072])
def test_select_random(wcc, P):
    rng = np.random.default_rng(P)
    nrm = (rng.random((3, P)) ** 4 * 100).astype(np.float32)
    for k in sorted({1, 2, P // 7 + 1, P // 2, P - 1, P}):
        _check_select(wcc, nrm, k)


@pytest.mark.parametrize("N,P", [(2, 200000), (10, 200000)])
def test_select_large_images_other_code_paths(wcc, N, P):
    """More keys per image than one cluster holds: the cooperative single kernel (few CTAs) and the one-kernel-per-phase
    path (more CTAs than can be resident at once)."""
    rng = np.random.default_rng(N)
    nrm = (rng.random((N, P)) ** 3).astype(np.float32)
    nrm[:, ::7] = nrm[:, 3:4]                                         # a long run of equal norms per image
    for k in (1, 70000, P - 5):
        _check_select(wcc, nrm, k)


def test_select_ties_and_special_values(wcc):
    rng = np.random.default_rng(3)
    P = 6000
    nrm = rng.integers(0, 4, size=(2, P)).astype(np.float32)          # long runs of equal norms
    for k in (1, 17, 1500, 3000, 4501, 5999, 6000):
        _check_select(wcc, nrm, k)
    _check_select(wcc, np.ones((1, 4096), np.float32), 100)            # all equal: the first k positions
    _check_select(wcc, np.zeros((2, 300), np.float32), 7)
    mixed = rng.standard_normal((2, 3000)).astype(np.float32)          # negative values and both zeros
    mixed[:, ::5] = 0.0
    mixed[:, 1::5] = -0.0
    for k in (10, 1200, 1900, 2999):
        _check_select(wcc, mixed, k)
    tiny = np.array([[1e-38, 3e-39, 1e-45, 0, 2e-38, 1e-45, 5e-39, 1e-38]], np.float32)    # subnormals
    for k in range(1, 9):
        _check_select(wcc, tiny, k)
    close = (1.0 + np.arange(4096) * 2.0 ** -23).astype(np.float32)[None]                 # differ in the last bits only
    close = close[:, rng.permutation(4096)].copy()
    for k in (1, 100, 2048, 4095):
        _check_select(wcc, close, k)


def test_select_on_real_norms(wcc):
    w = inputs.make("C1")
    coef, nrm2 = wcc.haar_fwd(torch.from_numpy(w.x).cuda(), w.levels)
    idx, tau = wcc.select_topk(nrm2, w.k)
    widx, wtau = oracle.select_topk(nrm2.cpu().numpy(), w.k)
    assert np.array_equal(idx.cpu().numpy(), widx) and np.array_equal(tau.cpu().numpy(), wtau)


def test_device_errors_are_reported_not_raised(wcc):
    x = torch.zeros((1, 1, 12, 8), device="cuda")
    with pytest.raises(wcc.WccError) as e:
        wcc.haar_fwd(x, 3)
    assert e.value.code == 2
    with pytest.raises(wcc.WccError) as e:
        wcc.select_topk(torch.zeros((1, 10), device="cuda"), 11)
    assert e.value.code == 3

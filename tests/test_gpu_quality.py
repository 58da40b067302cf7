"""The compression-quality sweep (Fig. 1 of the paper on synthetic maps): the GPU numbers equal the oracle's, fewer
bits on the int8 path match the oracle at full size, and the curve has the paper's shape (error falls with the bit
rate; shrinkage at 8 bits beats plain quantization at low rates on smooth maps)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2205_12268_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mods():
    from paper_2205_12268_b200 import build, wcc as w, quality as q
    build.build()
    assert torch.cuda.is_available()
    w.lib()
    return w, q


def _rel_mse(a, ref):
    d = a.astype(np.float64) - ref.astype(np.float64)
    return float((d * d).mean() / (ref.astype(np.float64) ** 2).mean())


def test_sweep_equals_the_oracle_on_a_small_map(mods):
    wcc, q = mods
    w = inputs.custom("quality", 40, 2, 16, 16, 64, 128, "f32", 3, 0.25, 8, n_sin=8, fmax=4.0)
    x = torch.from_numpy(w.x).cuda()
    rows = q.sweep(x, 3)
    eye = np.eye(16, dtype=np.float32)
    xmax = np.float32(w.x.max())
    prev = None
    for row in rows:
        r = row["effective_bits"]
        k = inputs.keep_count(r / 8.0, w.P)
        want = _rel_mse(oracle.forward(w.x, eye, 3, k, 8), w.x)
        assert abs(row["wcc_8bit_shrunk"] - want) <= 1e-9 + 1e-6 * want
        if r >= 2:
            want_b = _rel_mse(oracle.forward(w.x, eye, 3, w.P, r), w.x)
            assert abs(row["wcc_all_kept_rbit"] - want_b) <= 1e-9 + 1e-6 * want_b
        levels = np.float32((1 << r) - 1)
        std = xmax * np.round(levels * np.clip(w.x / xmax, 0, 1)) / levels          # Eq. 1-2, unsigned, by numpy
        assert abs(row["standard_rbit"] - _rel_mse(std, w.x)) <= 1e-6 * row["standard_rbit"]
        if prev is not None:
            assert row["wcc_8bit_shrunk"] <= prev                                   # keeping more never hurts
        prev = row["wcc_8bit_shrunk"]
    low = rows[1]
    assert low["effective_bits"] == 2 and low["wcc_8bit_shrunk"] < low["standard_rbit"]
    assert wcc.last_status() == 0


@pytest.mark.parametrize("bits", [2, 3, 5, 7])
@pytest.mark.parametrize("name", ["C4", "C5a"])
def test_fewer_bits_at_full_size(mods, name, bits):
    wcc, _ = mods
    w = inputs.make(name)
    x = torch.from_numpy(w.x.view(np.int16)).cuda().view(torch.bfloat16) if w.dtype == "bf16" else torch.from_numpy(w.x).cuda()
    y = wcc.forward(x, torch.from_numpy(w.Wt).cuda(), w.levels, w.k, bits)
    want = oracle.forward(w.x_f32(), w.Wt, w.levels, w.k, bits, out_bf16=(w.dtype == "bf16"))
    assert wcc.last_status() == 0
    assert np.array_equal(y.float().cpu().numpy().view(np.uint32), want.view(np.uint32))

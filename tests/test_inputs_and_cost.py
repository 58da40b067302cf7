"""The seeded generator (bytes only) and the App. D cost figures."""
import os

import numpy as np
import torch

from oracle import cost
from paper_2205_12268_b200 import inputs


def test_generator_is_deterministic_and_seeded():
    a = inputs.make("C1")
    b = inputs.make("C1")
    assert np.array_equal(a.x, b.x) and np.array_equal(a.Wt, b.Wt)
    c = inputs.make("C1", seed=1)
    assert not np.array_equal(a.x, c.x)
    assert a.x.shape == (1, 32, 64, 64) and a.x.dtype == np.float32 and a.k == 1024 and a.levels == 2


def test_counter_streams_are_position_addressable():
    full = inputs.uniform01(5, 3, 0, 100)
    assert np.array_equal(full[40:60], inputs.uniform01(5, 3, 40, 20))
    assert not np.array_equal(full, inputs.uniform01(5, 4, 0, 100))
    assert full.min() >= 0 and full.max() < 1
    z = inputs.normal(0, 9, 0, 200000)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1) < 0.01


def test_feature_map_statistics():
    x = inputs.feature_map(0, 1, 4, 64, 64, n_sin=8, fmax=4.0)
    assert (x < -0.3).sum() == 0                       # ReLU floor, only the 0.05 noise goes below zero
    flat = x[x < 0.02]
    assert flat.size > 1000 and 0.03 < flat.std() < 0.07
    w = inputs.weights(0, 256, 144)
    assert abs(w.std() * np.sqrt(144) - 1) < 0.02


def test_bf16_rounding_matches_library():
    a = (np.random.default_rng(0).standard_normal(10000) * 5).astype(np.float32)
    bits = inputs.f32_to_bf16_bits(a)
    want = torch.from_numpy(a).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, want)
    assert np.array_equal(inputs.bf16_bits_to_f32(bits), torch.from_numpy(a).to(torch.bfloat16).float().numpy())


def test_keep_counts_of_the_named_workloads():
    want = {"C1": 1024, "C2": 16384, "C3": 32768, "C4": 3840, "C4b": 1920, "C5a": 32768}
    for name, k in want.items():
        N, Cin, Cout, H, W, dtype, L, gamma, bits, s, f = inputs.CONFIGS[name]
        assert inputs.keep_count(gamma, H * W) == k
        assert H % (1 << L) == 0 and W % (1 << L) == 0
    assert inputs.keep_count(0.3, 10) == 3 and inputs.keep_count(0.31, 10) == 4


def test_bops_worked_example(golden_dir):
    g = {}
    with open(os.path.join(golden_dir, "appD_bops_example.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                key, val = line.split()
                g[key] = int(val)
    conv = cost.conv_bops(g["cin"], g["cout"], g["nw"], g["nh"], g["bits_w"], g["bits_a"])
    haar = cost.haar_bops(g["cin"], g["nw"], g["nh"], g["levels"], g["bits_a"]) + \
        cost.haar_bops(g["cout"], g["nw"], g["nh"], g["levels"], g["bits_a"])
    assert round(conv / 1e6) == g["conv_mbops"]
    assert round(haar / 1e6) == g["haar_mbops"]

"""Compression quality of the WCC activation path on synthetic maps: MSE against the effective bit rate.

The experiment behind Fig. 1 of the paper, on the seeded synthetic feature maps that stand in for its ImageNet
activations: an activation map is compressed by the layer's own pipeline (Haar transform, joint shrinkage to a fraction
gamma of the positions, 8-bit quantization, zero fill, inverse transform -- the layer with identity weights) and
compared with the original; the effective bit rate is 8 * gamma (Sec. 5, first experiment).  Beside it: plain uniform
quantization of the same map to b bits (Eq. 1-2, the unsigned case the paper uses for post-ReLU activations).

    python -m paper_2205_12268_b200.quality [--workload C2] [--levels 3]

Every WCC number comes from the CUDA library (wcc_forward through the binding); torch is only used to subtract and
average.  Prints one JSON object.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import inputs
from . import wcc


def compress_map(x: torch.Tensor, levels: int, gamma: float, bits: int = 8) -> torch.Tensor:
    """x [N][C][H][W] -> its reconstruction after shrinkage to ceil(gamma * H * W) positions and `bits`-bit codes."""
    N, Cc, H, W = x.shape
    eye = torch.eye(Cc, dtype=torch.float32, device=x.device)
    return wcc.forward(x, eye, levels, inputs.keep_count(gamma, H * W), bits)


def standard_quantization(x: torch.Tensor, b: int) -> torch.Tensor:
    """Uniform b-bit quantization of a non-negative map with the clipping parameter at its maximum (Eq. 1-2, unsigned):
    alpha * round((2^b - 1) * clip(x / alpha, 0, 1)) / (2^b - 1), computed in fp32."""
    xf = x.float()
    alpha = xf.max()
    levels_ = float((1 << b) - 1)
    return alpha * torch.round(levels_ * torch.clamp(xf / alpha, 0.0, 1.0)) / levels_


def relative_mse(a: torch.Tensor, ref: torch.Tensor) -> float:
    d = a.double() - ref.double()
    return float((d * d).mean() / (ref.double() * ref.double()).mean())


def sweep(x: torch.Tensor, levels: int = 3, rates=(1, 2, 3, 4, 5, 6, 7, 8)):
    """For every effective bit rate r: relative MSE of WCC at gamma = r / 8 (8-bit codes) and of r-bit uniform
    quantization; also WCC with every position kept and b = r bits (quantization of the wavelet coefficients alone)."""
    rows = []
    for r in rates:
        row = {"effective_bits": r, "wcc_8bit_shrunk": relative_mse(compress_map(x, levels, r / 8.0, 8), x)}
        if r >= 2:
            row["wcc_all_kept_rbit"] = relative_mse(compress_map(x, levels, 1.0, r), x)
        row["standard_rbit"] = relative_mse(standard_quantization(x, r), x)
        rows.append(row)
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="C2")
    ap.add_argument("--levels", type=int, default=0)
    args = ap.parse_args()
    w = inputs.make(args.workload)
    dev = torch.device("cuda", 0)
    if w.dtype == "bf16":
        x = torch.from_numpy(w.x.view(np.int16)).view(torch.bfloat16).to(dev)
    else:
        x = torch.from_numpy(w.x).to(dev)
    L = args.levels or w.levels
    out = {"workload": w.name, "shape": [w.N, w.Cin, w.H, w.W], "dtype": w.dtype, "levels": L,
           "metric": "mean squared error / mean square of the map", "rows": sweep(x, L)}
    assert wcc.last_status() == 0
    print(json.dumps(out))


if __name__ == "__main__":
    main()

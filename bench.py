#!/usr/bin/env python
"""Benchmark of the WCC layer forward pass (output Gpix/s) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C2] [--impl ours|reference]

A step is one pass of the whole layer (transform + norms, top-k select, gather + quantize, tensor-core
contraction, dequantize + scatter + inverse) over one synthetic batch.  Prints ONE JSON line.
With --gpus N > 1 (under torchrun) every rank runs the same-size batch of its own (weak scaling, no
data-path collective: images are independent and each rank's call uses its own activation scale).
--impl reference times the CPU oracle on the host cores instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "WCC layer output Gpix/s"
UNIT = "Gpix/s"
FLUSH_BYTES = 256 << 20          # > 126 MB of L2
STAGE_FILES = ("haar.cuh", "select.cuh", "gather.cuh", "regather.cuh", "contract.cuh", "fused.cuh", "fused_tiles.cuh", "tma.cuh",
               "libwcc.cu", "common.cuh")

# DRAM bytes per launch of the dominant kernel from one ncu capture (dram__bytes_read.sum + dram__bytes_write.sum),
# keyed by (workload, stage); valid only while the kernel sources still hash to `src`.
NCU_TRAFFIC = {
    # dram__bytes_read.sum + dram__bytes_write.sum of one launch, from the ncu captures summarised under profiles/.
    # C4 was captured with N=24 images (x = 189 MB > L2) and is divided by 2, C2 with N=16 and divided by 4: every stage
    # is per image, so traffic grows in proportion to the batch.
    ("C4", "fused_pass2"): {"bytes": (191781376 + 134613504) / 2, "src": "cde0b5a6e295"},
    ("C4", "haar_norms"): {"bytes": (189183744 + 3707392) / 2, "src": "cde0b5a6e295"},
    ("C2", "fused_pass2"): {"bytes": (153168896 + 13833984) / 4, "src": "cde0b5a6e295"},
    ("C2", "haar_norms"): {"bytes": (151312384 + 4362752) / 4, "src": "cde0b5a6e295"},
}


def _source_hash() -> str:
    h = hashlib.sha256()
    for f in STAGE_FILES:
        with open(os.path.join(ROOT, "paper_2205_12268_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:12]


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def stage_bytes(w, stage: str) -> float:
    """Algorithmic bytes one launch of a stage must move (what it reads once plus what it writes once)."""
    s = 2 if w.dtype == "bf16" else 4
    NP, Nk = w.N * w.P, w.N * w.k
    es = 2 if w.bits == 0 else 1
    return {
        "clear": w.N * (65536 + 3 * 2048) * 4,                                  # the select's histograms, zeroed (a memset node)
        "haar_norms": NP * w.Cin * s + 8 * NP + 5 * w.Cout * w.Cin,             # x once; norms and per-position max out; weights
        "fused_pass2": NP * w.Cin * s + 4 * NP + s * NP * w.Cout,               # x again, norms (or rank map), y once
        "haar_fwd_norms": NP * w.Cin * (s + 4) + 4 * NP,
        "select_topk": 4 * NP + 4 * Nk,
        "weight_quant": w.Cout * w.Cin * (4 + es),
        "gather_quant": 4 * Nk + 4 * Nk * w.Cin + es * Nk * w.Cin,
        "contract": es * Nk * w.Cin + es * w.Cin * w.Cout + 4 * Nk * w.Cout,
        "scatter_inv": 4 * Nk * w.Cout + 4 * Nk + s * NP * w.Cout,
    }[stage]


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int, period: float = 0.001):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.sm_max = [], set(), None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.nv = None

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
                 "hw_power_brake": 0x80, "sync_boost": 0x10}
        while not self._halt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for n, bit in names.items():
                    if r & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._halt.set()
        if self.is_alive():
            self.join(timeout=2)
        return {"sm_mhz": (statistics.median(self.samples) if self.samples else None), "sm_max_mhz": self.sm_max,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def _physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ------------------------------------------------------------------------------------------------ reference arm
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    from paper_2205_12268_b200 import inputs

    oracle.build()
    N, Cin, Cout, H, W, dtype, L, gamma, bits, n_sin, fmax = inputs.CONFIGS[args.workload]
    w = inputs.make(args.workload)
    x = w.x_f32()
    t0 = time.perf_counter()
    oracle.forward(x, w.Wt, L, w.k, bits, out_bf16=(dtype == "bf16"))
    t_full = time.perf_counter() - t0
    # bounded sample: shrink to whole images, then to a band of rows, until K+W steps fit ~2 minutes
    budget = 120.0 / max(1, args.steps + args.warmup)
    n_s, h_s = N, H
    while t_full * (n_s * h_s) / (N * H) > budget and n_s > 1:
        n_s = max(1, n_s // 2)
    while t_full * (n_s * h_s) / (N * H) > budget and h_s // 2 >= (1 << L) and (h_s // 2) % (1 << L) == 0:
        h_s //= 2
    xs = x[:n_s, :, :h_s, :].copy()
    k_s = inputs.keep_count(gamma, h_s * W)
    for _ in range(args.warmup):
        oracle.forward(xs, w.Wt, L, k_s, bits, out_bf16=(dtype == "bf16"))
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.forward(xs, w.Wt, L, k_s, bits, out_bf16=(dtype == "bf16"))
    dt = (time.perf_counter() - t0) / max(1, args.steps)
    val = n_s * h_s * W / dt / 1e9
    sample = "N=%d of %d images, %d of %d rows per step" % (n_s, N, h_s, H)
    out = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f32 transform, int8 x int8 -> int32 contraction", "data": "synthetic",
           "config": _config_dict(w, args, sample=sample),
           "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
           "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))
    return 0


def _config_dict(w, args, **extra):
    d = {"workload": "%s: N=%d Cin=%d Cout=%d H=%d W=%d %s levels=%d k=%d (%.4g of positions) bits=%d" % (
        w.name, w.N, w.Cin, w.Cout, w.H, w.W, w.dtype, w.levels, w.k, w.k / w.P, w.bits),
        "per_gpu_batch": w.N, "global_batch": w.N * args.gpus, "parallelism": "batch-sharded replicas x%d" % args.gpus}
    d.update(extra)
    return d


# ------------------------------------------------------------------------------------------------ multi-rank helpers
def rank_seed(rank: int) -> int:
    """Rank r draws its own batch of the workload's shape: seed 0 on rank 0 (the named workload), r elsewhere."""
    return rank


def max_over_ranks(dist, ms: float, device) -> float:
    """Device time of the slowest rank (the job is done when the last rank is)."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gpix(world: int, pixels_per_rank: int, ms_per_step: float) -> float:
    """Output pixels of all ranks per second, in Gpix/s (weak scaling: every rank processes pixels_per_rank)."""
    return world * pixels_per_rank / (ms_per_step * 1e-3) / 1e9


# ------------------------------------------------------------------------------------------------ our arm
L2_BYTES = 126 << 20
NOMINAL_HBM_GBS = 8000.0
CONTEXT_WORKLOADS = ("C1", "C2", "C3", "C3u", "C4", "C4b", "C5a", "C5b")


def layer_bytes(w):
    """Compulsory bytes of one layer (x once, y once) and the two-pass bound (the selection forces a second look at
    x; norms and per-position maxima written once and read once)."""
    s = 2 if w.dtype == "bf16" else 4
    NP = w.N * w.P
    b_min = s * NP * (w.Cin + w.Cout)
    return b_min, b_min + s * NP * w.Cin + 8 * NP


class Case:
    """One workload resident on the device: buffers, workspace, and the CUDA graph of one wcc_forward."""

    def __init__(self, wcc, torch, np, w, dev, staged=False, graph=True):
        self.wcc, self.torch, self.w, self.staged = wcc, torch, w, staged
        if w.dtype == "bf16":
            self.x_host = torch.from_numpy(w.x.view(np.int16)).view(torch.bfloat16).pin_memory()
        else:
            self.x_host = torch.from_numpy(w.x).pin_memory()
        self.x = self.x_host.to(dev)
        self.Wt = torch.from_numpy(w.Wt).to(dev)
        self.y = torch.empty((w.N, w.Cout, w.H, w.W), dtype=self.x.dtype, device=dev)
        self.y_host = torch.empty(self.y.shape, dtype=self.y.dtype).pin_memory()
        self.ws = wcc.Workspace.for_problem(self.x, w.Cout, w.levels, w.k, w.bits, staged=staged)
        self.pixels = w.N * w.H * w.W
        l0 = wcc.kernel_launches()
        self.eager()                                    # sets kernel attributes, counts launches
        self.launches_per_step = wcc.kernel_launches() - l0
        torch.cuda.synchronize()
        assert wcc.last_status() == 0
        self.graph = None
        if graph:
            try:
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    self.eager()
                torch.cuda.current_stream().wait_stream(side)
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    self.eager()
                self.graph = g
            except Exception as e:                      # keep going eagerly, and say so
                print("graph capture failed, timing eager launches: %r" % (e,), file=sys.stderr)
                self.graph = None
                torch.cuda.synchronize()
        self.step = self.graph.replay if self.graph is not None else self.eager

    def eager(self):
        w = self.w
        self.wcc.forward(self.x, self.Wt, w.levels, w.k, w.bits, y=self.y, ws=self.ws, staged=self.staged)

    def e2e(self):
        w = self.w
        self.x.copy_(self.x_host, non_blocking=True)
        self.wcc.forward(self.x, self.Wt, w.levels, w.k, w.bits, y=self.y, ws=self.ws, staged=self.staged)
        self.y_host.copy_(self.y, non_blocking=True)

    def e2e_overlapped(self, steps):
        """`steps` end-to-end steps as a serving loop would run them: two device buffers per direction and three streams,
        so that the upload of step i+1 and the download of step i-1 overlap the layer of step i.  Every step still
        uploads its input from pinned host memory and downloads its output.  Returns the device time of the whole loop."""
        torch, w = self.torch, self.w
        cur, up, down = torch.cuda.current_stream(), torch.cuda.Stream(), torch.cuda.Stream()
        xs, ys = [self.x, torch.empty_like(self.x)], [self.y, torch.empty_like(self.y)]
        arrived = [torch.cuda.Event() for _ in range(2)]
        computed = [torch.cuda.Event() for _ in range(2)]
        left = [torch.cuda.Event() for _ in range(2)]
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t0.record(cur)
        up.wait_event(t0)
        for i in range(steps):
            b = i & 1
            with torch.cuda.stream(up):
                if i >= 2:
                    up.wait_event(computed[b])          # the layer that read this buffer two steps ago is done
                xs[b].copy_(self.x_host, non_blocking=True)
                arrived[b].record(up)
            cur.wait_event(arrived[b])
            if i >= 2:
                cur.wait_event(left[b])                 # the output buffer has been downloaded
            self.wcc.forward(xs[b], self.Wt, w.levels, w.k, w.bits, y=ys[b], ws=self.ws, staged=self.staged)
            computed[b].record(cur)
            with torch.cuda.stream(down):
                down.wait_event(computed[b])
                self.y_host.copy_(ys[b], non_blocking=True)
                left[b].record(down)
        cur.wait_stream(up)
        cur.wait_stream(down)
        t1.record(cur)
        torch.cuda.synchronize()
        return t0.elapsed_time(t1)

    def stage_times(self, flush, steps):
        """Mean device time of every stage, from CUDA events recorded inside eager calls (L2 flushed before each)."""
        wcc = self.wcc
        names = wcc.STAGES if self.staged else wcc.FUSED_STAGES
        acc = [0.0] * len(wcc.STAGES)
        wcc.profile_enable(True)
        for _ in range(steps):
            flush.fill_(1)
            self.eager()
            for i, v in enumerate(wcc.profile_read()):
                acc[i] += v
        wcc.profile_enable(False)
        return {n: acc[i] / steps for i, n in enumerate(names)}


def chain_context(wcc, torch, np, inputs, dev, flush, peak, use_graph, steps=100):
    """The six-layer chain workload 32 -> 192 -> 32 ... with ReLU between the layers (2 x 256 x 512, bf16), every point of
    the sweep levels {1,2,3} x keep ratio {1/2,1/4,1/8,1/16}: one wcc_chain_forward per step (a CUDA graph replay, L2
    flushed before every step), beside the dense 1x1 bf16 chain (library matmul + ReLU) as the keep-everything reference."""
    N, H, W = 2, 256, 512
    chans = [32, 192, 32, 192, 32, 192, 32]
    first = inputs.custom("C5", 0, N, 32, 192, H, W, "bf16", 3, 0.25, 8, n_sin=16, fmax=8.0)
    x = torch.from_numpy(first.x.view(np.int16)).view(torch.bfloat16).to(dev)
    Ws = [torch.from_numpy(inputs.weights(100 + i, chans[i + 1], chans[i])).to(dev) for i in range(6)]
    y = torch.empty((N, 32, H, W), dtype=torch.bfloat16, device=dev)
    P = H * W
    b_min = sum(2 * N * P * (chans[i] + chans[i + 1]) for i in range(6))           # every layer: input once, output once

    def timed(fn, n):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        for a, b in ev:
            flush.fill_(1)
            a.record()
            fn()
            b.record()
        torch.cuda.synchronize()
        t = [a.elapsed_time(b) for a, b in ev]
        return sum(t) / len(t)

    def graphed(fn):
        fn()
        torch.cuda.synchronize()
        if not use_graph:
            return fn
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()
        torch.cuda.current_stream().wait_stream(side)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        return g.replay

    Wb = [w.to(torch.bfloat16) for w in Ws]

    def dense():
        cur = x.reshape(N, 32, P)
        for i in range(6):
            cur = torch.matmul(Wb[i], cur)
            if i < 5:
                cur = torch.relu_(cur)
        return cur

    dense_ms = timed(graphed(dense), steps)
    out = {"workload": "C5 chain: 6 layers 32->192->32..., ReLU between, N=2 H=256 W=512 bf16, bits=8",
           "compulsory_bytes": b_min, "dense_1x1_bf16_chain_ms": dense_ms, "steps": steps, "sweep": {}}
    for L in (1, 2, 3):
        for gamma in (0.5, 0.25, 0.125, 0.0625):
            k = inputs.keep_count(gamma, P)
            ch = wcc.Chain(x, Ws, L, k, 8)
            t = timed(graphed(lambda: ch(x, y)), steps)
            out["sweep"]["L%d_g%s" % (L, gamma)] = {
                "levels": L, "keep": gamma, "k": k, "ms": t, "Gpix/s_per_layer": 6 * N * P / (t * 1e-3) / 1e9,
                "frac_of_peak": b_min / (t * 1e-3) / 1e9 / peak, "frac_of_nominal_8TBs": b_min / (t * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
                "vs_dense_chain": t / dense_ms}
            del ch
    assert wcc.last_status() == 0
    return out


# (N, c_in, expansion, H, W, keep ratio): a few of the shapes of the paper's own GPU benchmark of the block (App. H, Table 8)
BLOCK_SHAPES = [(8, 512, 2, 96, 96, 0.25), (4, 256, 4, 128, 128, 0.25), (2, 256, 4, 256, 256, 0.125), (2, 128, 4, 128, 128, 0.25)]


def make_block(wcc, torch, inputs, dev, shape):
    N, Cc, e, H, W, gamma = shape
    E = Cc * e
    g = torch.Generator(device=dev).manual_seed(Cc + H)
    x = torch.relu(torch.randn((N, Cc, H, W), device=dev, generator=g)).to(torch.bfloat16)
    W1 = torch.randn((E, Cc), device=dev, generator=g) / Cc ** 0.5
    W3 = torch.randn((Cc, E), device=dev, generator=g) / E ** 0.5
    Wdw = torch.randn((E, 3, 3), device=dev, generator=g) / 3
    blk = wcc.Block(x, W1, Wdw, W3, 3, inputs.keep_count(gamma, H * W), 8)
    return x, W1, Wdw, W3, blk


def block_context(wcc, torch, np, inputs, dev, flush, steps=30):
    """The inverted residual block of the paper's own GPU benchmark, y = x + K3(Kdw(K1 x)) with both pointwise
    convolutions as WCC layers (three levels, 8 bits) at a few of its shapes, beside the same block with dense bf16
    library kernels (matmul, grouped conv2d).  Batches are smaller than the paper's (its batches filled an 11 GB card)."""
    import torch.nn.functional as F
    out = []
    for shape in BLOCK_SHAPES:
        N, Cc, e, H, W, gamma = shape
        E = Cc * e
        x, W1, Wdw, W3, blk = make_block(wcc, torch, inputs, dev, shape)
        y = torch.empty_like(x)

        def timed(fn):
            # both arms are captured once and replayed, as the headline layer is: neither pays for its launches
            fn()
            torch.cuda.synchronize()
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                fn()
            torch.cuda.current_stream().wait_stream(side)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                fn()
            ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
            for a, b in ev:
                flush.fill_(1)
                a.record()
                g.replay()
                b.record()
            torch.cuda.synchronize()
            t = [a.elapsed_time(b) for a, b in ev]
            del g
            return sum(t) / len(t)

        W1b, W3b, Wdwb = W1.to(torch.bfloat16), W3.to(torch.bfloat16), Wdw.to(torch.bfloat16)[:, None]

        def dense():
            u = torch.matmul(W1b, x.reshape(N, Cc, H * W)).reshape(N, E, H, W)
            v = F.conv2d(u, Wdwb, padding=1, groups=E)
            return x + torch.matmul(W3b, v.reshape(N, E, H * W)).reshape(N, Cc, H, W)

        t_wcc = timed(lambda: blk(x, y))
        t_dense = timed(dense)
        out.append({"N": N, "c": Cc, "expansion": e, "H": H, "W": W, "keep": gamma, "wcc_block_ms": t_wcc,
                    "dense_bf16_block_ms": t_dense, "dense_over_wcc": t_dense / t_wcc})
        del blk, x, y
        torch.cuda.empty_cache()
    assert wcc.last_status() == 0
    return out


def run_ours(args):
    import numpy as np
    import torch

    from paper_2205_12268_b200 import build as wbuild
    from paper_2205_12268_b200 import inputs
    from paper_2205_12268_b200 import wcc

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the oracle")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        wbuild.build()
    if dist:
        dist.barrier()
    wcc.lib()

    if args.workload.startswith("block"):               # profiling aid: one inverted residual block alone (eager launches)
        shape = BLOCK_SHAPES[int(args.workload[5:] or 0)]
        x, _, _, _, blk = make_block(wcc, torch, inputs, dev, shape)
        y = torch.empty_like(x)
        for _ in range(max(3, args.warmup) + args.steps):
            blk(x, y)
        torch.cuda.synchronize()
        assert wcc.last_status() == 0
        print(json.dumps({"workload": "inverted residual block N=%d c=%d e=%d %dx%d keep=%g" % shape, "lean": True}))
        return 0
    if args.workload == "C5chain":                      # profiling aid: the six-layer chain alone (three levels, keep 1/4)
        flush = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device=dev)
        peak, _ = _peaks()
        N, H, W = (args.batch or 2), 256, 512
        chans = [32, 192, 32, 192, 32, 192, 32]
        first = inputs.custom("C5", 0, N, 32, 192, H, W, "bf16", 3, 0.25, 8, n_sin=16, fmax=8.0)
        x = torch.from_numpy(first.x.view(np.int16)).view(torch.bfloat16).to(dev)
        Ws = [torch.from_numpy(inputs.weights(100 + i, chans[i + 1], chans[i])).to(dev) for i in range(6)]
        ch = wcc.Chain(x, Ws, 3, first.k, 8)
        y = torch.empty((N, 32, H, W), dtype=torch.bfloat16, device=dev)
        for _ in range(max(3, args.warmup)):
            flush.fill_(1)
            ch(x, y)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for a, b in ev:
            flush.fill_(1)
            a.record()
            ch(x, y)
            b.record()
        torch.cuda.synchronize()
        assert wcc.last_status() == 0
        t = sum(a.elapsed_time(b) for a, b in ev) / len(ev)
        print(json.dumps({"workload": "C5chain N=%d L=3 keep=0.25 (eager launches)" % N, "ms_per_chain": t, "lean": True}))
        return 0
    over = {"N": args.batch} if args.batch else {}
    w = inputs.make(args.workload, seed=rank_seed(rank), **over)
    case = Case(wcc, torch, np, w, dev, staged=args.staged, graph=not args.no_graph)
    flush = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device=dev)
    warmup = max(3, args.warmup)

    def timed_loop(fn, steps):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in ev:
            flush.fill_(1)                              # evict x, y and the scratch from L2
            a.record()
            fn()
            b.record()
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in ev]

    for _ in range(warmup):
        flush.fill_(1)
        case.step()
    torch.cuda.synchronize()

    sampler = ClockSampler(_physical_gpu_index(local_rank))
    sampler.start()
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    t_wall0 = time.perf_counter()
    ms = timed_loop(case.step, args.steps)
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    t_wall = time.perf_counter() - t_wall0
    n_timed_samples = len(sampler.samples)
    assert wcc.last_status() == 0
    total_ms = max_over_ranks(dist, float(sum(ms)), dev)
    ms_per_step = total_ms / args.steps
    value = whole_job_gpix(world, case.pixels, ms_per_step)

    if args.lean:                                       # profiling runs: the timed loop only
        sampler.stop()
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "ms_per_step": ms_per_step, "lean": True,
                              "config": _config_dict(w, args)}))
        if dist:
            dist.destroy_process_group()
        return 0

    # end to end through the public call: host input -> device, layer, device -> host output, every step
    e2e_steps = min(args.steps, 200)
    for _ in range(3):
        case.e2e()
    torch.cuda.synchronize()
    e_ms = timed_loop(case.e2e, e2e_steps)
    e_total = max_over_ranks(dist, float(sum(e_ms)), dev)
    e2e_serial = whole_job_gpix(world, case.pixels, e_total / e2e_steps)
    case.e2e_overlapped(4)
    e_total = max_over_ranks(dist, float(case.e2e_overlapped(e2e_steps)), dev)
    e2e_val = whole_job_gpix(world, case.pixels, e_total / e2e_steps)

    # per-stage device times with CUDA events recorded inside the call (eager launches of the same configuration)
    peak, peak_kind = _peaks()
    stage_ms = case.stage_times(flush, max(50, min(args.steps, 200)))
    dom = max((n for n in stage_ms if n != "clear"), key=stage_ms.get)      # a memset node is not one of our kernels
    achieved = stage_bytes(w, dom) / (stage_ms[dom] * 1e-3) / 1e9
    tr = NCU_TRAFFIC.get((w.name, dom))
    traffic = tr["bytes"] if tr and tr.get("src") == _source_hash() and not args.batch else None
    b_min, b_2p = layer_bytes(w)
    gbs = lambda nbytes, t_ms: nbytes / (t_ms * 1e-3) / 1e9
    x_bytes = (2 if w.dtype == "bf16" else 4) * w.N * w.P * w.Cin
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic, "peak_kind": "%s HBM copy bandwidth" % peak_kind,
                "algorithmic_bytes_per_launch": stage_bytes(w, dom),
                "stage_ms": stage_ms,
                "stage_frac_of_peak": {n: gbs(stage_bytes(w, n), stage_ms[n]) / peak for n in stage_ms if stage_ms[n] > 0},
                "x_fits_l2": x_bytes < L2_BYTES,
                "note": ("x (%.0f MB) is smaller than the 126 MB L2, so part of the second pass's re-read of x can be served "
                         "from L2: its fraction is algorithmic bytes over time, not DRAM throughput" % (x_bytes / 1e6))
                        if x_bytes < L2_BYTES else "x is larger than L2: both passes stream it from DRAM",
                "layer": {"compulsory_bytes": b_min, "two_pass_bytes": b_2p,
                          "frac_of_peak": gbs(b_min, ms_per_step) / peak,
                          "frac_of_two_pass_bound": gbs(b_2p, ms_per_step) / peak,
                          "frac_of_nominal_8TBs": gbs(b_min, ms_per_step) / NOMINAL_HBM_GBS,
                          "two_pass_frac_of_nominal_8TBs": gbs(b_2p, ms_per_step) / NOMINAL_HBM_GBS}}

    if rank != 0:
        sampler.stop()
        if dist:
            dist.destroy_process_group()
        return 0

    # dense 1x1 convolution on the uncompressed map (library kernel), for context
    def dense_ms_of(c):
        try:
            xd = c.x.reshape(c.w.N, c.w.Cin, c.w.P)
            Wd = c.Wt.to(c.x.dtype)
            torch.matmul(Wd, xd)
            return statistics.median(timed_loop(lambda: torch.matmul(Wd, xd), 50))
        except Exception:
            return None

    dense_ms = dense_ms_of(case)

    # every other workload, briefly: graph replay time, stage times, fractions (single GPU context, not the headline)
    workloads = {}
    if not args.batch and not args.no_context:
        ctx_steps = 200
        for name in CONTEXT_WORKLOADS:
            if name == w.name and not args.staged:
                c, c_ms = case, ms
            else:
                c = Case(wcc, torch, np, inputs.make(name), dev, graph=not args.no_graph)
                for _ in range(3):
                    flush.fill_(1)
                    c.step()
                c_ms = timed_loop(c.step, ctx_steps)
            t = sum(c_ms) / len(c_ms)
            st = stage_ms if c is case else c.stage_times(flush, 100)
            bm, b2 = layer_bytes(c.w)
            workloads[name] = {
                "config": _config_dict(c.w, args)["workload"], "steps": len(c_ms), "ms_per_step": t,
                "Gpix/s": c.pixels / (t * 1e-3) / 1e9,
                "layer_frac_of_peak": gbs(bm, t) / peak, "layer_frac_of_two_pass_bound": gbs(b2, t) / peak,
                "layer_frac_of_nominal_8TBs": gbs(bm, t) / NOMINAL_HBM_GBS,
                "stage_ms": st,
                "stage_frac_of_peak": {n: gbs(stage_bytes(c.w, n), st[n]) / peak for n in st if st[n] > 0},
                "dense_1x1_matmul_ms": dense_ms if c is case else dense_ms_of(c),
                "x_fits_l2": (2 if c.w.dtype == "bf16" else 4) * c.w.N * c.w.P * c.w.Cin < L2_BYTES}
            if c is not case:
                del c
                torch.cuda.empty_cache()
        assert wcc.last_status() == 0
    chain = blocks = None
    if not args.batch and not args.no_context:
        chain = chain_context(wcc, torch, np, inputs, dev, flush, peak, not args.no_graph)
        blocks = block_context(wcc, torch, np, inputs, dev, flush)
    clocks_all = sampler.stop()
    timed = sampler.samples[:max(1, n_timed_samples)]
    clocks = {"sm_mhz": (statistics.median(timed) if timed else None), "sm_max_mhz": clocks_all["sm_max_mhz"],
              "reasons": clocks_all["reasons"], "samples": len(timed),
              "whole_run": {"sm_mhz": clocks_all["sm_mhz"], "samples": clocks_all["samples"]}}

    # the oracle on the host cores: a bounded sample of the same workload
    import oracle
    oracle.build()
    xo = w.x_f32()
    t0 = time.perf_counter()
    oracle.forward(xo, w.Wt, w.levels, w.k, w.bits, out_bf16=(w.dtype == "bf16"))
    t1 = time.perf_counter() - t0
    reps = max(1, min(200, int(10.0 / max(t1, 1e-3))))
    t0 = time.perf_counter()
    for _ in range(reps):
        oracle.forward(xo, w.Wt, w.levels, w.k, w.bits, out_bf16=(w.dtype == "bf16"))
    t_cpu = (time.perf_counter() - t0) / reps
    cpu = {"value": case.pixels / t_cpu / 1e9, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
           "sample": "the full workload, %d repetitions (%.1f s of CPU work)" % (reps, t_cpu * reps)}

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
           "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "f32 transform, int8 x int8 -> int32 contraction" if w.bits else "f32 transform, bf16 contraction",
           "data": "synthetic",
           "config": _config_dict(w, args, l2="flushed before every step by a %d MiB write outside the step's events" % (FLUSH_BYTES >> 20),
                                  launch=("CUDA graph replay of one %s" if case.graph is not None else "eager %s") % (
                                      "wcc_forward_staged" if args.staged else "wcc_forward"),
                                  wall_s_timed_region=t_wall),
           "clocks": clocks,
           "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": case.x_host.numel() * case.x_host.element_size(),
                   "d2h_bytes_per_step": case.y_host.numel() * case.y_host.element_size(), "steps": e2e_steps,
                   "how": "every step uploads its input from pinned host memory and downloads its output; the copies of "
                          "neighbouring steps overlap the layer (two device buffers, three streams)",
                   "one_step_at_a_time": e2e_serial},
           "gpu_launches": int(case.launches_per_step * args.steps),
           "roofline": roofline, "cpu_baseline": cpu,
           "context": {"dense_1x1_matmul_ms": dense_ms, "ms_per_step_median": statistics.median(ms),
                       "ms_per_step_min": min(ms), "workloads": workloads, "chain": chain, "inverted_residual_blocks": blocks}}
    print(json.dumps(out))
    if dist:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="C4")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="time eager wcc_forward calls instead of a graph replay")
    ap.add_argument("--batch", type=int, default=0, help="override the number of images per GPU")
    ap.add_argument("--lean", action="store_true", help="timed loop only (for runs under a profiler)")
    ap.add_argument("--no-context", action="store_true", help="skip the brief runs of the other workloads")
    ap.add_argument("--staged", action="store_true", help="time wcc_forward_staged (every intermediate in memory)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())

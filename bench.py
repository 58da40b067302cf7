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
STAGE_FILES = ("haar.cuh", "select.cuh", "gather.cuh", "contract.cuh", "fused.cuh", "fused_tiles.cuh", "tma.cuh", "libwcc.cu",
               "common.cuh")

# DRAM bytes per launch of the dominant kernel from one ncu capture (dram__bytes_read.sum + dram__bytes_write.sum),
# keyed by (workload, stage); valid only while the kernel sources still hash to `src`.
NCU_TRAFFIC = {
    # captured with N=16 images of C2 (x = 151 MB > L2) and divided by 4: every stage is per image
    ("C2", "fused_pass2"): {"bytes": (153168896 + 13174272) / 4, "src": "858dc5d135d2"},
    ("C2", "haar_norms"): {"bytes": (151201536 + 4285184) / 4, "src": "858dc5d135d2"},
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

    def __init__(self, index: int, period: float = 0.005):
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

    over = {"N": args.batch} if args.batch else {}
    w = inputs.make(args.workload, seed=rank_seed(rank), **over)
    if w.dtype == "bf16":
        x_host = torch.from_numpy(w.x.view(np.int16)).view(torch.bfloat16).pin_memory()
    else:
        x_host = torch.from_numpy(w.x).pin_memory()
    x = x_host.to(dev)
    Wt = torch.from_numpy(w.Wt).to(dev)
    y = torch.empty((w.N, w.Cout, w.H, w.W), dtype=x.dtype, device=dev)
    y_host = torch.empty(y.shape, dtype=y.dtype).pin_memory()
    ws = wcc.Workspace.for_problem(x, w.Cout, w.levels, w.k, w.bits, staged=args.staged)
    flush = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device=dev)
    pixels = w.N * w.H * w.W

    def step_eager():
        wcc.forward(x, Wt, w.levels, w.k, w.bits, y=y, ws=ws, staged=args.staged)

    # one eager call first: sets kernel attributes, counts launches
    l0 = wcc.kernel_launches()
    step_eager()
    launches_per_step = wcc.kernel_launches() - l0
    torch.cuda.synchronize()
    assert wcc.last_status() == 0

    graph = None
    if not args.no_graph:
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                step_eager()
            torch.cuda.current_stream().wait_stream(side)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                step_eager()
            graph = g
        except Exception as e:                          # keep going eagerly, and say so
            print("graph capture failed, timing eager launches: %r" % (e,), file=sys.stderr)
            graph = None
            torch.cuda.synchronize()
    step = graph.replay if graph is not None else step_eager

    def timed_loop(fn, steps, pre=None):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in ev:
            flush.fill_(1)                              # evict x, y and the scratch from L2
            if pre:
                pre()
            a.record()
            fn()
            b.record()
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in ev]

    for _ in range(max(3, args.warmup)):
        flush.fill_(1)
        step()
    torch.cuda.synchronize()

    sampler = ClockSampler(_physical_gpu_index(local_rank))
    sampler.start()
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    t_wall0 = time.perf_counter()
    ms = timed_loop(step, args.steps)
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    t_wall = time.perf_counter() - t_wall0
    clocks = sampler.stop()
    assert wcc.last_status() == 0
    total_ms = max_over_ranks(dist, float(sum(ms)), dev)
    ms_per_step = total_ms / args.steps
    value = whole_job_gpix(world, pixels, ms_per_step)

    if args.lean:                                       # profiling runs: the timed loop only
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "ms_per_step": ms_per_step, "lean": True,
                              "config": _config_dict(w, args)}))
        if dist:
            dist.destroy_process_group()
        return 0

    # end to end through the public call: host input -> device, layer, device -> host output, every step
    def e2e_step():
        x.copy_(x_host, non_blocking=True)
        wcc.forward(x, Wt, w.levels, w.k, w.bits, y=y, ws=ws, staged=args.staged)
        y_host.copy_(y, non_blocking=True)

    e2e_steps = min(args.steps, 200)
    for _ in range(3):
        e2e_step()
    torch.cuda.synchronize()
    e_ms = timed_loop(e2e_step, e2e_steps)
    e_total = max_over_ranks(dist, float(sum(e_ms)), dev)
    e2e_val = whole_job_gpix(world, pixels, e_total / e2e_steps)

    # per-stage device times with CUDA events recorded inside the call, same launch configuration (eager)
    wcc.profile_enable(True)
    prof_steps = min(args.steps, 200)
    names = wcc.STAGES if args.staged else wcc.FUSED_STAGES
    acc = [0.0] * len(wcc.STAGES)
    for _ in range(prof_steps):
        flush.fill_(1)
        step_eager()
        for i, v in enumerate(wcc.profile_read()):
            acc[i] += v
    wcc.profile_enable(False)
    stage_ms = {n: acc[i] / prof_steps for i, n in enumerate(names)}
    dom = max((n for n in stage_ms if n != "clear"), key=stage_ms.get)      # the memset node is not one of our kernels
    peak, peak_kind = _peaks()
    achieved = stage_bytes(w, dom) / (stage_ms[dom] * 1e-3) / 1e9
    tr = NCU_TRAFFIC.get((w.name, dom))
    traffic = tr["bytes"] if tr and tr.get("src") == _source_hash() else None
    layer_min_bytes = (2 if w.dtype == "bf16" else 4) * w.N * w.P * (w.Cin + w.Cout)
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic, "peak_kind": "%s HBM copy bandwidth" % peak_kind,
                "algorithmic_bytes_per_launch": stage_bytes(w, dom),
                "stage_ms": stage_ms,
                "stage_frac_of_peak": {n: stage_bytes(w, n) / (stage_ms[n] * 1e-3) / 1e9 / peak for n in stage_ms},
                "layer": {"compulsory_bytes": layer_min_bytes,
                          "frac_of_peak": layer_min_bytes / (ms_per_step * 1e-3) / 1e9 / peak}}

    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return 0

    # dense 1x1 convolution on the uncompressed map (library kernel), for context
    dense_ms = None
    try:
        xd = x.reshape(w.N, w.Cin, w.P)
        Wd = Wt.to(x.dtype)
        torch.matmul(Wd, xd)
        dense_ms = statistics.median(timed_loop(lambda: torch.matmul(Wd, xd), 50))
    except Exception:
        pass

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
    cpu = {"value": pixels / t_cpu / 1e9, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
           "sample": "the full workload, %d repetitions (%.1f s of CPU work)" % (reps, t_cpu * reps)}

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
           "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "f32 transform, int8 x int8 -> int32 contraction" if w.bits else "f32 transform, bf16 contraction",
           "data": "synthetic",
           "config": _config_dict(w, args, l2="flushed before every step by a %d MiB write outside the step's events" % (FLUSH_BYTES >> 20),
                                  launch=("CUDA graph replay of one %s" if graph is not None else "eager %s") % (
                                      "wcc_forward_staged" if args.staged else "wcc_forward"),
                                  wall_s_timed_region=t_wall),
           "clocks": clocks,
           "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": x_host.numel() * x_host.element_size(),
                   "d2h_bytes_per_step": y_host.numel() * y_host.element_size(), "steps": e2e_steps},
           "gpu_launches": int(launches_per_step * args.steps),
           "roofline": roofline, "cpu_baseline": cpu,
           "context": {"dense_1x1_matmul_ms": dense_ms, "ms_per_step_median": statistics.median(ms),
                       "ms_per_step_min": min(ms)}}
    print(json.dumps(out))
    if dist:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="C2")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="time eager wcc_forward calls instead of a graph replay")
    ap.add_argument("--batch", type=int, default=0, help="override the number of images per GPU")
    ap.add_argument("--lean", action="store_true", help="timed loop only (for runs under a profiler)")
    ap.add_argument("--staged", action="store_true", help="time wcc_forward_staged (every intermediate in memory)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())

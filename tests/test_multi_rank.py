"""The N > 1 harness logic on CPU: two gloo ranks on 127.0.0.1 (no GPU, no kernels)."""
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2205_12268_b200 import inputs
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # every rank times its own batch; the job's time is the slowest rank's
    slowest = bench.max_over_ranks(dist, 10.0 + 5.0 * rank, torch.device("cpu"))
    # batches are sharded by rank: same shape, different draws, no exchange
    w = inputs.custom("shard", bench.rank_seed(rank), 1, 3, 3, 8, 8, "f32", 1, 0.5, 8)
    sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(sums, torch.tensor([float(w.x.sum())], dtype=torch.float64))
    dist.barrier()
    out.put((rank, slowest, [float(s) for s in sums], tuple(w.x.shape)))
    dist.destroy_process_group()


def test_two_ranks_max_time_and_sharded_batches():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, sums, shape in res:
        assert slowest == 15.0                       # max over ranks, seen by both
        assert shape == (1, 3, 8, 8)
        assert sums[0] != sums[1]                    # each rank drew its own batch
    assert res[0][2] == res[1][2]


def test_whole_job_value_is_the_sum_over_ranks():
    sys.path.insert(0, ROOT)
    import bench
    one = bench.whole_job_gpix(1, 131072, 0.1)
    assert abs(one - 1.31072) < 1e-9
    assert abs(bench.whole_job_gpix(8, 131072, 0.1) - 8 * one) < 1e-9


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""

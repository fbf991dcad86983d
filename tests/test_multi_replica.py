"""The path does not shard across GPUs (replicas only): with N ranks the benchmark runs N independent
replicas, takes the MAX of the per-rank step times and reports the aggregate.  That host logic is
exercised here with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, e2e = bench.max_over_ranks([10.0 + rank, 20.0 - rank])
    dist.barrier()
    if rank == 0:
        out.put((ms, e2e, bench.aggregate_value(2, 5, ms, world)))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_aggregate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    ms, e2e, value = res
    assert ms == 11.0 and e2e == 20.0
    assert abs(value - 2 * 2 * 5 / 0.011) < 1e-6


def test_single_process_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.aggregate_value(2, 40, 50.0, 1) == 1600.0


def test_gpus_flag_must_agree_with_the_launched_world_size():
    """`--gpus N` means N replicas: under a launcher whose WORLD_SIZE differs the script refuses to run
    (exit code 2) instead of silently timing another number of replicas."""
    import subprocess
    env = dict(os.environ, WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")
    for impl in ("ours", "reference"):
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", impl, "--steps", "1"],
                           env=env, capture_output=True, text=True, timeout=120)
        assert r.returncode == 2 and "WORLD_SIZE" in r.stderr, (impl, r.returncode, r.stderr[-300:])

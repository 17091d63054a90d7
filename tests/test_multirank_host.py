"""Host-side logic of the multi-GPU bench path, exercised with two gloo ranks on the CPU.

This library has no exchange between GPUs: N ranks are N independent replicas, each with its
own data stream; the only collective is the maximum of the timings over the ranks."""
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2509_05679_b200 import synth as sy
    net = sy.config(0)
    x = sy.batch_inputs(net, 0, stream=rank)                 # every replica draws its own data stream
    ms, e2e = bench.max_over_ranks([10.0 + 5.0 * rank, 1.0 + rank], dist, "cpu")
    out.put((rank, ms, e2e, float(x.ravel()[0])))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_maximum_time_and_draw_different_data():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0] and [r[2] for r in res] == [2.0, 2.0]
    assert res[0][3] != res[1][3]
    import bench
    # whole-job value: both replicas' samples over the slowest replica's time
    assert bench.whole_job_throughput(1024, 10, 2, 0.015 * 10) == 1024 * 10 * 2 / 0.15


def test_reference_arm_is_silent_on_ranks_other_than_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""

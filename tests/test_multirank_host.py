"""The N > 1 path of the bench on CPU: two gloo ranks.  The layer shards by (stream, head) with
no exchange inside it, so ranks are independent replicas; what the ranks share is the timing
protocol (max over ranks) and distinct input seeds."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2605_16579_b200 import workload

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local = [10.0 + rank, 3.0 - rank, 0.5 * (rank + 1)]
    got = bench.max_over_ranks(local, world, torch.device("cpu"))
    seeds, blk = bench.rank_seeds(rank)
    cfg = workload.custom(B=1, H=2, D=64, L=32)
    q, _, _, _ = workload.step_inputs(cfg, 0, seeds[0])
    dist.barrier()
    out[rank] = (got, seeds, blk, float(q.double().sum()))
    dist.destroy_process_group()


def test_two_ranks_max_and_distinct_inputs():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        r0, r1 = out[0], out[1]
    assert r0[0] == r1[0] == [11.0, 3.0, 1.0]          # every rank sees the slowest rank's times
    assert set(r0[1]).isdisjoint(r1[1]) and r0[2] != r1[2]
    assert r0[3] != r1[3]                                # replicas work on different data


def test_whole_job_value_scales_with_replicas():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2605_16579_b200 import workload

    cfg = workload.CONFIGS["long"]
    one = bench.whole_job_value(cfg, 1, 2.0)
    assert abs(one - cfg.B * cfg.L * cfg.steps / 2e-3) < 1e-6
    assert abs(bench.whole_job_value(cfg, 8, 2.0) - 8 * one) < 1e-3
    assert bench.max_over_ranks([1.5, 2.5], 1, None) == [1.5, 2.5]


def test_gpus_flag_starts_that_many_ranks():
    """`--gpus N` outside a launcher starts N ranks itself; inside one it must agree with it."""
    import subprocess

    sys.path.insert(0, ROOT)
    import bench

    cmd = bench.launcher_command(4, ["--gpus", "4", "--steps", "2"], port=29777)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"]
    assert "--nproc-per-node=4" in cmd and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "2"] and cmd[-5].endswith("bench.py")
    env = dict(os.environ, WORLD_SIZE="2", RANK="0", LOCAL_RANK="0")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "1"], env=env,
                         capture_output=True, text=True, timeout=120)
    assert out.returncode != 0 and "WORLD_SIZE=2" in out.stderr

"""World-size-2 check (gloo, CPU) of the benchmark's multi-rank bookkeeping: ranks are independent
replicas, the only exchange is the MAX over ranks of the timed intervals, rank 0 reports the sum of
the replicas' images/s.  Also the reference arm: rank 0 alone prints its line, other ranks stay silent."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import torch
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [10.0 + 5 * rank, 2.0 - rank]          # rank 1 is slower on the first interval, faster on the second
    red = bench.max_over_ranks(mine, torch.device("cpu"), world)
    out[rank] = red
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_with_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    with ctx.Manager() as mgr:
        out = mgr.dict()
        procs = [ctx.Process(target=_worker, args=(r, 2, 29611, out)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(120)
            assert p.exitcode == 0
        assert out[0] == [15.0, 2.0] and out[1] == [15.0, 2.0]


def test_whole_job_value_is_the_sum_of_replicas():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.whole_job_value(8, 1, 2.0) == 4000.0
    assert bench.whole_job_value(8, 4, 2.0) == 16000.0
    assert bench.max_over_ranks([1.5, 2.5], None, 1) == [1.5, 2.5]


def test_reference_arm_prints_one_line_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0",
                        "--workload", "layer32"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0",
                        "--workload", "layer32", "--gpus", "2"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["config"]["workload"] == "layer32"

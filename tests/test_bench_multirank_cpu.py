"""The N > 1 path of the benchmark is "replicas only": ranks share nothing on the data path and only agree on
the slowest rank's time.  That agreement (barrier + MAX all-reduce) and the whole-job throughput arithmetic are
checked here with two gloo ranks on the CPU; so is the reference arm's rule that only rank 0 works."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))     # rank 1 is the slow one
    out[rank] = (ms, bench.whole_job_value(1000, world, ms, steps=2))
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value_gloo():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29731, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 15.0
    assert abs(res[0][1] - 2 * 1000 / (15.0e-3 / 2)) < 1e-6
    assert bench.max_over_ranks(7.5) == 7.5


def test_step_flops_matches_scope_table():
    from paper_2203_17189_b200 import workloads as WL
    want = {"small": 6.785, "base": 54.43, "xl": 170.95, "declm": 130.16}
    for name, tf in want.items():
        assert abs(bench.step_flops(WL.model_dims(name)) / 1e12 - tf) < 0.01 * tf


def test_reference_arm_only_rank0_prints():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"

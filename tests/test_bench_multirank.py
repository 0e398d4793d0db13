"""The N > 1 leg of bench.py ("replicas only": every rank runs the whole step on its own GPU, no
data-path collective): the timing reduction is a MAX over ranks and the value counts all ranks'
units.  Exercised with world_size 2 on the gloo backend (CPU)."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, ms_e2e = bench.max_over_ranks([10.0 + 5 * rank, 40.0 - 3 * rank], "cpu")
    dist.barrier()
    if rank == 0:
        json.dump({"ms": ms, "ms_e2e": ms_e2e,
                   "value": bench.whole_job_value(world, 1000, 4, ms)}, open(out, "w"))
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value(tmp_path):
    out = str(tmp_path / "r0.json")
    mp.spawn(_worker, args=(2, 29531 + os.getpid() % 200, out), nprocs=2, join=True)
    r = json.load(open(out))
    assert r["ms"] == 15.0 and r["ms_e2e"] == 40.0          # slowest rank of each figure
    assert abs(r["value"] - 2 * 1000 * 4 / 15e-3) < 1e-6    # both ranks' units over the slowest time


def test_single_process_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], "cpu") == [1.5, 2.5]


def test_reference_arm_prints_only_on_rank_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "linear_fp32"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0 and p.stdout.strip() == ""
    env["RANK"] = "0"
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "linear_fp32"],
                       env=env, capture_output=True, text=True, timeout=300)
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0

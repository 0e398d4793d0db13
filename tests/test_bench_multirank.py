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


class _WallStamp:
    """CPU stand-in for the CUDA event bench.py stamps its timed region with."""
    def __init__(self):
        import time
        self.t = time.perf_counter()

    def elapsed_time(self, later):
        return 1e3 * (later.t - self.t)


def _region_worker(rank, world, port, out):
    import time
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    calls = []

    def step(i):                                  # rank 1 is the slow one
        calls.append(i)
        time.sleep(0.02 * (1 + 2 * rank))

    ms = bench.timed_region(step, 4, dist.barrier, _WallStamp)
    (slowest,) = bench.max_over_ranks([ms], "cpu")
    if rank == 0:
        json.dump({"own": ms, "slowest": slowest, "calls": calls,
                   "value": bench.whole_job_value(world, 1000, 4, slowest)}, open(out, "w"))
    dist.barrier()
    dist.destroy_process_group()


def test_timed_region_under_two_ranks(tmp_path):
    """The timed region of the benchmark (barrier, exactly K steps, barrier) with two gloo ranks of
    different speed: rank 0 reports the slow rank's time and both ranks' units."""
    out = str(tmp_path / "r0.json")
    mp.spawn(_region_worker, args=(2, 29331 + os.getpid() % 200, out), nprocs=2, join=True)
    r = json.load(open(out))
    assert r["calls"] == [0, 1, 2, 3]
    assert 80 <= r["own"] < 200 and 240 <= r["slowest"] < 600      # 4 x 20 ms against 4 x 60 ms
    assert abs(r["value"] - 2 * 1000 * 4 / (r["slowest"] * 1e-3)) < 1e-6


def test_gpus_flag_starts_that_many_ranks():
    """`bench.py --gpus N` outside a launcher starts N ranks itself (one process per GPU, loopback
    rendezvous).  Without a CUDA device every rank must refuse loudly: there is no CPU fallback."""
    import torch
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.rank_command(3, ["--gpus", "3", "--steps", "2"])
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=3" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[-4:] == ["--gpus", "3", "--steps", "2"]
    assert os.path.samefile(cmd[cmd.index("--master-port") + 2], os.path.join(ROOT, "bench.py"))
    if torch.cuda.is_available():
        return
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1",
                        "--workload", "linear_fp32", "--no-cpu-baseline"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert p.returncode != 0
    assert p.stderr.count("bench.py needs a CUDA device") >= 2      # both ranks were started and refused


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

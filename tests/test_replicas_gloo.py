"""The multi-rank host logic of the benchmark, on CPU with the gloo backend.

With more than one GPU every rank steps an independent replica (the path has no
exchange step between GPUs), the reported time is the slowest rank's and the
value counts the elements of all ranks.  Two gloo processes stand in for two GPUs."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.rank_env() == (rank, world, rank)
    my_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow replica
    ms = bench.max_over_ranks(my_ms, world, torch.device("cpu"))
    value = bench.job_value(1000, 4, world, ms)
    dist.barrier()
    if rank == 0:
        torch.save({"ms": ms, "value": value}, out)
    dist.destroy_process_group()


def test_two_replicas_report_slowest_time_and_total_elements(tmp_path):
    out = str(tmp_path / "r0.pt")
    mp.spawn(_rank_main, args=(2, _free_port(), out), nprocs=2, join=True)
    got = torch.load(out)
    assert got["ms"] == 15.0
    assert abs(got["value"] - 2 * 1000 * 4 / 15e-3) < 1e-6


def test_single_rank_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, 1, torch.device("cpu")) == 7.5
    assert bench.job_value(10, 2, 1, 1000.0) == 20.0


def test_reference_arm_runs_on_rank_zero_only(tmp_path):
    import subprocess
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                        "--gpus", "2", "--steps", "1", "--warmup", "0", "--workload", "flat20",
                        "--sample-log2", "12"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                        "--gpus", "2", "--steps", "1", "--warmup", "0", "--workload", "flat20",
                        "--sample-log2", "12"], env=env, capture_output=True, text=True, timeout=120)
    import json
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0

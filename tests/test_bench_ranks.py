"""Host logic of bench.py for more than one rank, on CPU with gloo: the timing
is the slowest rank's, the value counts every replica's units, and the CPU
reference arm runs on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    local_ms = 10.0 if rank == 0 else 14.0
    ms = bench.max_over_ranks(local_ms)
    val = bench.whole_job_value(1000, world, 7, ms)
    with open(out % rank, "w") as f:
        json.dump({"ms": ms, "value": val}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_slowest_time_and_whole_job_units(tmp_path):
    out = str(tmp_path / "r%d.json")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    for r in range(2):
        got = json.load(open(out % r))
        assert got["ms"] == 14.0
        assert abs(got["value"] - 2 * 1000 * 7 / 0.014) < 1e-6


def test_single_process_needs_no_group():
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_value(10, 1, 2, 1000.0) == 20.0


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "C1",
                        "--steps", "1", "--warmup", "0", "--gpus", "2"], env=env, capture_output=True, text=True)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = env["LOCAL_RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "C1",
                        "--steps", "2", "--warmup", "1", "--gpus", "2"], env=env, capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": line["unit"], "h2d_bytes_per_step": 0,
                           "d2h_bytes_per_step": 0}

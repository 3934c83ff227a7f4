"""The benchmark's whole-job arithmetic on two ranks (gloo, CPU): time = MAX over ranks, units add up;
and its reference arm leaves every rank but 0 silent."""
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 10.0 if rank == 0 else 25.0          # rank 1 is the slow one
    ms, value = bench.whole_job(ms_local, units_per_rank=1000.0, dist=dist)
    out[rank] = (ms, value)
    dist.barrier()
    dist.destroy_process_group()


def test_whole_job_takes_max_time_and_sums_units():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        ms, value = res[rank]
        assert ms == 25.0
        assert abs(value - 2 * 1000.0 / 25e-3) < 1e-6


def test_whole_job_single_process():
    import bench
    ms, value = bench.whole_job(4.0, 8.0)
    assert ms == 4.0 and value == 8.0 / 4e-3


def test_reference_arm_prints_only_on_rank_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "small",
                        "--steps", "3", "--warmup", "3"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "small",
                        "--steps", "3", "--warmup", "3", "--gpus", "2"], env=env, capture_output=True, text=True, timeout=300)
    import json
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0

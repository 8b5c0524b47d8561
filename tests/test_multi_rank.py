"""The N > 1 leg of bench.py on CPU: two gloo ranks run the aggregation the
benchmark uses (whole-job units = sum over ranks, time = max over ranks) and the
reference arm's rule that only rank 0 prints.  The data path has no collective:
every rank runs the same batch shape on its own device."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, rank, world)
    # rank r processed 100*(r+1) units in 10*(r+1) ms
    units, ms = bench.aggregate(100.0 * (rank + 1), 10.0 * (rank + 1), "cpu")
    dist.barrier()
    with open(os.path.join(out_dir, "r%d.json" % rank), "w") as f:
        json.dump({"units": units, "ms": ms}, f)
    dist.destroy_process_group()


def test_aggregate_sum_of_units_max_of_time_two_gloo_ranks(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for r in range(2):
        got = json.load(open(tmp_path / ("r%d.json" % r)))
        assert got == {"units": 300.0, "ms": 20.0}


def test_aggregate_is_identity_without_a_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert not dist.is_initialized()
    assert bench.aggregate(7.0, 3.0, "cpu") == (7.0, 3.0)


def test_reference_arm_prints_on_rank0_only():
    """`bench.py --impl reference` under a 2-rank launch: rank 1 exits 0 without output."""
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--gpus", "2", "--steps", "1", "--warmup", "0", "--config", "1"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode == 0 and res.stdout.strip() == ""
    env["RANK"] = "0"
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--gpus", "2", "--steps", "1", "--warmup", "0", "--config", "1"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode == 0
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0

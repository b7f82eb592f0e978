"""N > 1 reporting logic on CPU: two gloo ranks, rendezvous on 127.0.0.1."""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2107_14575_b200 import replicas

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str) -> None:
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert replicas.env_rank() == (rank, world, rank)
    local_ms = [3.0, 7.5][rank]                      # rank 1 is the slow one
    dist.barrier()
    ms = replicas.max_over_ranks(local_ms)
    rate = replicas.whole_job_rate(units_per_rank=1.0e6, world=world, ms=ms)
    # every rank holds the same answer; only rank 0 reports
    gathered = [None] * world
    dist.all_gather_object(gathered, (ms, rate))
    if rank == 0:
        with open(os.path.join(out_dir, "line.json"), "w") as fh:
            json.dump({"ms": ms, "rate": rate, "all": gathered}, fh)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_summed_work(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    rec = json.load(open(tmp_path / "line.json"))
    assert rec["ms"] == 7.5
    assert rec["rate"] == pytest.approx(2 * 1.0e6 / 7.5e-3)
    assert rec["all"][0] == rec["all"][1]


def test_single_process_passes_the_value_through():
    assert replicas.max_over_ranks(4.25) == 4.25
    assert replicas.whole_job_rate(10.0, 1, 1000.0) == 10.0


def test_reference_arm_prints_only_on_rank_zero():
    """Under a multi-rank launch the ranks other than 0 leave without work or output."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    env["LOCAL_RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["value"] > 0 and line["unit"] == "GB/s"

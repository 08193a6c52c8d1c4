"""Host logic of the benchmark's N > 1 path, on CPU with the gloo backend (world size 2): the
step time is the maximum over ranks, and only rank 0 of the reference arm prints."""
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
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    got = bench.reduce_max(10.0 + rank, world)
    dist.barrier()
    with open(os.path.join(out, f"r{rank}.json"), "w") as fh:
        json.dump({"max": got}, fh)
    dist.destroy_process_group()


def test_step_time_is_max_over_ranks(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        assert json.load(open(tmp_path / f"r{r}.json"))["max"] == 11.0


def test_reference_arm_prints_on_rank0_only():
    base = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "conv3x3",
            "--steps", "2", "--warmup", "1", "--gpus", "2"]
    env = dict(os.environ, WORLD_SIZE="2", MASTER_ADDR="127.0.0.1")
    r1 = subprocess.run(base, env=dict(env, RANK="1"), capture_output=True, text=True, timeout=300)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = subprocess.run(base, env=dict(env, RANK="0"), capture_output=True, text=True, timeout=300)
    assert r0.returncode == 0
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["n_gpus"] == 2
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert torch.__version__

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


def _probe(out):
    """What a spawned rank of bench.py sees: torchrun's variables, and a working rendezvous."""
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    assert os.environ["LOCAL_RANK"] == str(rank) and os.environ["MASTER_ADDR"] == "127.0.0.1"
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    got = bench.reduce_max(3.0 * (rank + 1), world)
    dist.barrier()
    with open(os.path.join(out, f"s{rank}.json"), "w") as fh:
        json.dump({"max": got, "world": world}, fh)
    dist.destroy_process_group()


def test_bench_starts_its_own_ranks_when_not_under_torchrun(tmp_path):
    """`bench.py --gpus N` outside torchrun spawns the N ranks itself (here: the spawn and the
    rendezvous, with gloo on CPU)."""
    import bench
    env = {k: os.environ.pop(k) for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_PORT") if k in os.environ}
    try:
        bench.spawn_ranks(2, _probe, str(tmp_path))
    finally:
        os.environ.update(env)
    for r in range(2):
        got = json.load(open(tmp_path / f"s{r}.json"))
        assert got == {"max": 6.0, "world": 2}


def test_reference_arm_spawned_prints_one_line():
    """--impl reference --gpus 2 outside torchrun: two ranks start, rank 0 alone prints."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "conv3x3",
                        "--steps", "2", "--warmup", "1", "--gpus", "2"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.strip().splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["dtype"] == "f32"


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

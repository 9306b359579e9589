"""Host logic of the multi-replica benchmark, on CPU with two gloo ranks.

The path does not shard, so N GPUs run N independent replicas; what the benchmark adds is the
reduction of the per-rank time to the slowest rank and the whole-job aggregate.  Also checks that the
reference arm prints on rank 0 only.
"""
import json
import os
import socket
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def worker(rank: int, world: int, port: int, out_dir: str):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    local_ms = 100.0 + 50.0 * rank                     # rank 1 is the slow one
    slow = bench.slowest_rank(local_ms, world, "cpu")
    value = bench.whole_job_throughput(1000, 2, world, slow)
    dist.barrier()
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"slow": slow, "value": value}, f)
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_add_their_work(tmp_path):
    world = 2
    mp.spawn(worker, args=(world, free_port(), str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        got = json.load(open(tmp_path / f"rank{rank}.json"))
        assert got["slow"] == 150.0
        assert abs(got["value"] - world * 1000 * 2 / 0.150) < 1e-6


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.slowest_rank(12.5, 1, "cpu") == 12.5
    assert bench.whole_job_throughput(10, 3, 1, 1000.0) == 30.0


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_gpus_flag_starts_that_many_ranks_by_itself(tmp_path):
    """`bench.py --gpus N` without a launcher starts N ranks with RANK / LOCAL_RANK / WORLD_SIZE set and a
    common rendezvous; here the ranks are a small CPU script that meets over gloo, so the spawning logic runs
    without a GPU.  And a rank count that differs from --gpus is refused."""
    sys.path.insert(0, ROOT)
    import bench
    script = tmp_path / "rank.py"
    script.write_text(
        "import json, os, sys\n"
        "import torch, torch.distributed as dist\n"
        "dist.init_process_group('gloo')\n"
        "t = torch.tensor([float(os.environ['RANK']) + 1.0])\n"
        "dist.all_reduce(t)\n"
        "json.dump({'rank': int(os.environ['RANK']), 'local': int(os.environ['LOCAL_RANK']),\n"
        "           'world': dist.get_world_size(), 'sum': float(t.item()), 'argv': sys.argv[1:]},\n"
        "          open(os.path.join(sys.argv[1], 'spawned%s.json' % os.environ['RANK']), 'w'))\n"
        "print('line from rank', os.environ['RANK'])\n"
        "dist.destroy_process_group()\n")
    rc = bench.spawn_replicas([str(tmp_path), "--gpus", "2"], 2, entry=[sys.executable, str(script)])
    assert rc == 0
    for rank in range(2):
        got = json.load(open(tmp_path / f"spawned{rank}.json"))
        assert got == {"rank": rank, "local": rank, "world": 2, "sum": 3.0, "argv": [str(tmp_path), "--gpus", "2"]}
    env = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--steps", "1"], env=env,
                         capture_output=True, text=True, timeout=120)
    assert out.returncode != 0 and "refusing" in out.stderr and out.stdout.strip() == ""

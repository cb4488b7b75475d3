"""The multi-rank side of bench.py on CPU: the path has no inter-GPU exchange, so N ranks are N
independent replicas and the only collective is the maximum of the per-rank times (gloo here,
NCCL on GPUs).  Also: the oracle arm prints from rank 0 only."""
import json
import os
import subprocess
import sys

import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r "measured" (10 + r) ms device-resident and (20 - r) ms end to end
    got = bench.max_over_ranks([10.0 + rank, 20.0 - rank], world, torch.device("cpu"))
    dist.barrier()
    dist.destroy_process_group()
    with open(os.path.join(out, f"rank{rank}.json"), "w") as f:
        json.dump(got, f)


def test_max_over_ranks_two_gloo_ranks(tmp_path):
    world = 2
    port = 29500 + os.getpid() % 1000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        got = json.load(open(tmp_path / f"rank{rank}.json"))
        assert got == [11.0, 20.0]          # the slowest rank of each measurement, on every rank


def test_whole_job_value_counts_every_replica():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.0], 1, None) == [3.0, 4.0]
    # two replicas of 98,304 transitions each, the slower one took 5 ms
    assert bench.whole_job_value(98304, 2, 5.0) == pytest.approx(2 * 98304 / 5e-3)


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_gpus_flag_starts_its_own_ranks():
    """Started plainly (no WORLD_SIZE), --gpus 2 runs the script again as two ranks under torch.distributed.run; on
    the oracle arm rank 0 alone works and prints ONE line, which names both ranks."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--workload",
                        "tiny", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["config"]["workload"] == "tiny"

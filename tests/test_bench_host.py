"""Host-side logic of bench.py: the CPU-baseline arm prints one well-formed line, ranks other than
0 stay silent, and the max-over-ranks / whole-job aggregation works across two gloo ranks."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, check=True, cwd=ROOT)
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["unit"] == "tokens/s" and rec["value"] > 0
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["cpu_baseline"]["cores"] >= 1
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["config"]["workload"] == "tiny"


def test_reference_arm_other_ranks_do_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny",
                          "--gpus", "2", "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env,
                         cwd=ROOT)
    assert out.returncode == 0 and out.stdout.strip() == ""


def _rank_main(rank, world, port, results):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 100.0 + 50.0 * rank                       # rank 1 is the slow one
    mx = bench.reduce_max(ms)
    results[rank] = (mx, bench.whole_job_tokens_per_s(world, 10, 256, mx))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation_gloo():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        results = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, results), nprocs=world, join=True)
        for r in range(world):
            mx, v = results[r]
            assert mx == 150.0
            assert abs(v - 2 * 10 * 256 / 0.150) < 1e-6


def test_single_process_is_identity():
    assert bench.reduce_max(12.5) == 12.5
    assert bench.whole_job_tokens_per_s(1, 10, 256, 1000.0) == 2560.0

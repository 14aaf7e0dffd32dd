"""The N > 1 path of bench.py on CPU: replicas only, no data-path collective.

Two gloo ranks each report a step time; the job's time is the slowest rank's and its
throughput the sum over ranks.  Also checks the reference arm's rank gating and the
algorithmic byte counts the benchmark divides by.
"""
import json
import os
import subprocess
import sys

import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2608_12932_b200 import workload as wl  # noqa: E402


def _rank_main(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    job_ms = bench.max_over_ranks(ms, dist, "cpu")
    value = bench.whole_job_gbs(1e6, 100, world, job_ms)
    dist.barrier()
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"job_ms": job_ms, "value": value}, f)
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_time_and_sum_the_work(tmp_path):
    world, port = 2, 29511 + os.getpid() % 500
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"r{r}.json")) for r in range(world)]
    assert res[0] == res[1]
    assert res[0]["job_ms"] == 15.0
    assert abs(res[0]["value"] - (1e6 * 100 * 2) / 15e-3 / 1e9) < 1e-9


def test_single_process_is_identity():
    assert bench.max_over_ranks(3.5, None, "cpu") == 3.5
    assert bench.whole_job_gbs(2e9, 1, 1, 1000.0) == 2.0


def test_reference_arm_only_runs_on_rank_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "3", "--gpus", "2"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_reference_arm_line_on_rank_zero():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                          "--warmup", "3"], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "GB/s" and line["steps"] == 2
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0


def test_algorithmic_bytes_match_the_definition():
    M, N, K = 8, 6144, 4096
    G = K // 128
    assert wl.algorithmic_bytes_gemm(M, N, K) == N * K // 2 + G * N * 2 + G * N // 2 + M * K + 2 * M + 4 * M * G + 2 * M * N
    assert wl.algorithmic_bytes_gemm(M, N, K) == 13206544
    assert wl.algorithmic_bytes_quantize(M, K) == 3 * M * K + 2 * M + 4 * M * G
    assert wl.algorithmic_ops(1024, 24576, 4096) == 2 * 1024 * 24576 * 4096
